#!/usr/bin/env python
"""Benchmark of the token-mask hot path.

One step = one decode step of the whole batch: accept the previously sampled tokens, build every
request's next-token bitmask (cached sets merged with the Earley check of the uncertain tokens),
apply it to the batch's logits in place.  The workload is the seeded synthetic config C3
(128 requests, each with its own JSON-schema grammar, vocabulary 151 936, bf16 logits) unless
--workload says otherwise.  Grammar compilation (cache build) is timed once before the steps and
reported beside them.

Prints one JSON line.  `--impl reference` times the CPU oracle instead, as it stands, on a
bounded sample of the same workload.
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

from paper_2601_04426_b200 import inputs  # noqa: E402

SHAPES = {"C1": (1, 8192), "C2": (1, 128256), "C3": (128, 151936), "C4": (64, 128256), "C5": (256, 200064),
          "T5": (16, 128256), "T20": (16, 128256), "T50": (16, 128256), "T100": (16, 128256),
          "H16": (32, 128256), "H64": (32, 128256), "P10": (8, 128256), "P100": (8, 128256), "P500": (8, 128256), "R256": (16, 128256), "R1024": (16, 128256), "R4096": (16, 128256)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons (read-only NVML queries, every millisecond) while the
    measured passes run; falls back to polling nvidia-smi if the NVML binding is missing."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int = 0):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.reasons = set()
        self.stop_flag = threading.Event()
        self.max_mhz = None
        self.proc = None

    def run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.index
            if visible:
                try:
                    phys = int(visible.split(",")[self.index])
                except ValueError:
                    phys = self.index
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self.stop_flag.is_set():
                self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                bits = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
                time.sleep(0.001)
            return
        except Exception:
            pass
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + q, "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.proc.stdout:
            if self.stop_flag.is_set():
                break
            parts = [x.strip() for x in line.split(",")]
            try:
                self.samples.append(float(parts[0]))
                self.max_mhz = float(parts[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    self.reasons.add(n)

    def finish(self):
        self.stop_flag.set()
        if self.proc is not None:
            self.proc.terminate()       # the exact child started above
        self.join(timeout=2.0)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        sm = sorted(self.samples)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(sm)}


def oracle_leg(w, steps, warmup, threads=None, n_req=None, budget_s=25.0):
    """The CPU oracle, as it stands, on a bounded sample: the masks of the first requests of the batch along
    their trajectories plus the apply of one row each, scaled to a whole batch step.  The same (request, step)
    pairs whatever arm calls it, so the figures of the two arms can be compared."""
    from oracle import oracle as O
    from oracle import schema_ebnf as SE
    threads = threads or O.default_threads()
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    n_req = min(w.batch, len(w.request_grammar), n_req or 16)
    oms = [O.Matcher(O.Grammar(SE.grammar_text(w.grammars[w.request_grammar[b]].kind, w.grammars[w.request_grammar[b]].text))) for b in range(n_req)]
    logits = inputs.make_logits(w.logits_seed, 1, w.vocab.size, w.dtype)
    per_step = []
    t_begin = time.perf_counter()
    for step in range(min(warmup + steps, w.steps)):
        t0 = time.perf_counter()
        for b in range(n_req):
            mask = oms[b].mask(ov, threads)
            O.apply_mask(logits, mask[None, :])
        dt = time.perf_counter() - t0
        for b in range(n_req):
            tok = w.trajectories[b][step]
            if oms[b].accept_token(ov, tok) == 2:
                oms[b].reset()
        if step >= warmup:
            per_step.append(dt / n_req * w.batch)
        if time.perf_counter() - t_begin > budget_s and len(per_step) >= 1:
            break
    us = 1e6 * float(np.mean(per_step))
    sample = "steps %d..%d x the first %d of %d requests (mask + apply of each), scaled x%.1f to the batch" % (
        warmup, warmup + len(per_step) - 1, n_req, w.batch, w.batch / n_req)
    return us, threads, sample


def oracle_cache_build_leg(w, n_scannable_total, threads, n_positions=48, budget_s=10.0):
    """The oracle's classification (accepted / uncertain / rejected of every token at one scannable state,
    from the flattened tables) on a seeded sample of positions of the first grammar, extrapolated to the
    workload's scannable positions."""
    from oracle import oracle as O
    from paper_2601_04426_b200 import binding as XB
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    g = XB.Grammar(None, w.grammars[0].kind, w.grammars[0].text)          # host front end only: the tables
    t = g.tables()
    scal = {k: t.pop(k) for k in ("n_rules", "n_states", "n_classes", "root_rule", "root_nullable")}
    tb = O.Tables(scal["n_rules"], scal["n_states"], scal["n_classes"], scal["root_rule"], scal["root_nullable"], **t)
    states = tb.scannable_states()
    rng = inputs.Rng(inputs.config_seed(w.name) ^ 0xB111D)
    picked = [states[rng.below(len(states))] for _ in range(min(n_positions, len(states)))]
    t0 = time.perf_counter()
    done = 0
    for st in picked:
        tb.classify(ov, st, threads)
        done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    g.close()
    pairs_per_s = done * w.vocab.size / dt
    return {"pairs_per_s": pairs_per_s, "seconds_extrapolated": n_scannable_total * w.vocab.size / pairs_per_s, "cores": threads,
            "sample": "%d seeded positions of grammar 0 x the whole vocabulary, extrapolated to %d scannable positions" % (done, n_scannable_total)}


def kernels_sha():
    """First 16 hex digits of the SHA-256 of the kernel source: ncu figures are tied to the kernels they were taken on."""
    import hashlib
    with open(os.path.join(ROOT, "paper_2601_04426_b200", "csrc", "kernels.cuh"), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def ncu_figures(workload, batch):
    """Counters read from ncu captures (profiles/ncu_counters.json), or {} when they were taken on another
    version of the kernels or on another workload."""
    path = os.path.join(ROOT, "profiles", "ncu_counters.json")
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        rec = json.load(f)
    if rec.get("kernels_sha16") != kernels_sha():
        return {}
    return rec.get("workloads", {}).get("%s/%d" % (workload, batch), {})


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3", choices=sorted(SHAPES))
    ap.add_argument("--batch", type=int, default=None, help="shrink the batch (debugging only; the line then names it)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--step", default="three", choices=["three", "fill_apply", "accept_fill"],
                    help="how a step is launched: 'three' = fill, apply, accept as three launches (default); 'fill_apply' = fill and apply "
                         "in one launch, then accept; 'accept_fill' = apply, then accept and the next mask's fill in one launch")
    ap.add_argument("--jit-sweep", default=None,
                    help="comma-separated K values (or 'full'): compile just in time with K entries precomputed and report "
                         "compile time and per-step time avg / P99 / max over the trajectory (the shape of the paper's K sweep)")
    ap.add_argument("--compile-threads", type=int, default=0, help="host threads compiling the grammars (0 = one per core, at most 16)")
    ap.add_argument("--repeat-threshold", type=int, default=0,
                    help="bounded repetitions of at least this many iterations keep a count in the Earley item (Section 3.6); "
                         "0 = the library's default (64), -1 = expand every repetition into explicit states")
    ap.add_argument("--no-state-compression", action="store_true",
                    help="build one cache entry per scannable state (ablation of the repetition state compression)")
    args = ap.parse_args()
    warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    B0, V = SHAPES[args.workload]
    metric = "per-step token-mask us (accept + fill + apply) at batch %d x vocab %d" % (args.batch or B0, V)

    if args.impl == "reference":
        if rank != 0:
            return 0
        w = inputs.make_workload(args.workload, batch=min(args.batch or B0, 16))
        w_full_batch = args.batch or B0
        us, threads, sample = oracle_leg(_with_batch(w, w_full_batch), args.steps, args.warmup)
        line = {"impl": "reference", "metric": metric, "value": us, "unit": "us/step", "n_gpus": args.gpus, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
                "dtype": "int32", "data": "synthetic", "config": {"workload": args.workload, "batch": w_full_batch, "vocab": V},
                "cpu_baseline": {"value": us, "unit": "us/step", "cores": threads, "kind": "oracle", "sample": sample},
                "e2e": {"value": us, "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    import torch
    from paper_2601_04426_b200 import binding as XB
    from paper_2601_04426_b200 import dist_util, engine
    torch.cuda.set_device(local_rank)
    dist_util.init_from_env("nccl")
    XB.lib()          # fails loudly if the CUDA library is missing

    w = inputs.make_workload(args.workload, batch=args.batch)
    if args.jit_sweep:
        if rank == 0:
            print(json.dumps(jit_sweep(w, args, local_rank)))
        dist_util.finish()
        return 0
    if world > 1:     # weak scaling: every rank serves its own batch of requests (no data-path collective)
        w = dist_util.rotate_requests(w, rank)
    # one small compile first, so that the reported build time holds no context creation or lazy module loading
    wt = XB.Tokenizer([bytes([i]) for i in range(256)] + [b""], 256, [])
    XB.Grammar(wt, "ebnf", 'root ::= [a-z]+ "."').close()
    wt.close()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    s = engine.Session(w, device="cuda:%d" % local_rank, state_compression=not args.no_state_compression, compile_threads=args.compile_threads,
                       repeat_threshold=args.repeat_threshold)
    torch.cuda.synchronize()
    session_s = time.perf_counter() - t0
    compile_s = s.compile_wall_s
    stats = [g.stats() for g in s.grammars]
    pool_reserved = s.pool.stats()["reserved_bytes"]
    build_ms = sum(x["cache_build_ms"] for x in stats)
    pairs = sum(x["pairs_classified"] for x in stats)
    pairs_dense = sum(x["n_scannable"] for x in stats) * s.V

    n, W = s.n, s.W
    elt = 2 if w.dtype == "bf16" else 4
    tdtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    # logits ring larger than twice the L2, so the apply kernel always works out of HBM
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size
    bytes_one = n * s.V * elt
    ring_n = max(2, int(np.ceil(2.2 * l2 / bytes_one)) + 1)
    base = engine.logits_tensor(inputs.make_logits(w.logits_seed, min(n, 8), s.V, w.dtype), s.device)
    ring = [base.repeat((n + base.shape[0] - 1) // base.shape[0], 1)[:n].contiguous() for _ in range(ring_n)]
    traj = torch.from_numpy(np.asarray([[w.trajectories[b][t] for b in range(n)] for t in range(w.steps)], dtype=np.int32)).to(s.device)      # [steps, n]
    total = warmup + args.steps
    launches = {"accept": 0, "fill": 0, "apply": 0, "reset": 0, "accept_fill": 0, "fill_apply": 0}      # this library's kernels only

    # The decode loop is launch-bound (short kernels), so the timed loop replays CUDA graphs, as a
    # serving engine's decode loop does: one graph per trajectory step, with the step's token ids
    # read straight from the resident trajectory table and the logits buffer taken from the ring.
    # Every way of launching a step runs accept, fill and apply once for every request; a request
    # that accepts end of sequence starts its next document in the accept launch.
    #   three        fill, apply, accept                                      (3 launches, the default)
    #   fill_apply   fill + apply in one launch, accept                       (2 launches)
    #   accept_fill  apply, accept + fill of the next mask in one launch      (2 launches; needs a first fill)
    #   no_apply     fill, accept: not a step -- the three-launch step without its apply, for apply's in-step cost
    def body_of(mode):
        def body(buf, t):
            if mode == "fill_apply":
                s.fill_apply(buf)
                s.accept_device(traj[t], restart_on_eos=True)
            elif mode == "three":
                s.fill(); s.apply(buf)
                s.accept_device(traj[t], restart_on_eos=True)
            elif mode == "accept_fill":
                s.apply(buf)
                s.accept_fill_device(traj[t], restart_on_eos=True)
            else:
                s.fill()
                s.accept_device(traj[t], restart_on_eos=True)
        return body

    per_step_launches = {"fill_apply": {"fill_apply": 1, "accept": 1}, "three": {"fill": 1, "apply": 1, "accept": 1},
                         "accept_fill": {"apply": 1, "accept_fill": 1}, "no_apply": {"fill": 1, "accept": 1}}

    def restart(mode):
        for b in range(n):
            s.reset(b)
        launches["reset"] += n
        if mode == "accept_fill":
            s.fill()
            launches["fill"] += 1

    def capture(mode, group=1):
        """One graph per `group` consecutive trajectory steps."""
        body = body_of(mode)
        restart(mode)
        torch.cuda.synchronize()
        graphs = []
        for t0_ in range(0, w.steps - group + 1, group):
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph):
                for t in range(t0_, t0_ + group):
                    body(ring[t % ring_n], t)
            graphs.append(gph)
        torch.cuda.synchronize()
        return graphs

    def replay_pass(mode, graphs, n_replays, n_warm, group=1, count=False):
        """Replays graph i % len(graphs) for i in [0, n_warm + n_replays); returns us per step of the last n_replays."""
        restart(mode)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(n_warm + n_replays):
            if i == n_warm:
                if count:
                    for k in launches:
                        launches[k] = 0
                dist_util.barrier()
                torch.cuda.synchronize()
                e0.record()
            if i % len(graphs) == 0 and i > 0:
                restart(mode)
            graphs[i % len(graphs)].replay()
            for k, c in per_step_launches[mode].items():
                launches[k] += c * group
        e1.record()
        torch.cuda.synchronize()
        dist_util.barrier()
        return dist_util.max_over_ranks(e0.elapsed_time(e1)) * 1e3 / (n_replays * group)

    for mode in ("three", "fill_apply", "accept_fill"):      # eager warm-up of every call before capture (first-use set-up)
        restart(mode)
        for k in range(ring_n):
            body_of(mode)(ring[k], 0)
    torch.cuda.synchronize()

    # ---- pass A: the headline number (events only around the timed region) --------------------
    sampler = ClockSampler(local_rank)
    sampler.start()
    graphs = capture(args.step)
    us_per_step = replay_pass(args.step, graphs, args.steps, warmup, count=True)
    timed_launches = sum(launches.values())
    del graphs

    # ---- the same steps launched the other ways, and eight steps per graph (context, not the headline) ------
    # A serving engine's decode graph holds the model's forward pass too, so the launch of the
    # graph is shared with everything else in the step.  With eight steps per graph, seven of
    # eight step boundaries are kernel-to-kernel edges like the ones inside a step.
    by_mode = {args.step: us_per_step}
    for mode in ("fill_apply", "three", "accept_fill", "no_apply"):
        if mode not in by_mode:
            g2 = capture(mode)
            by_mode[mode] = replay_pass(mode, g2, args.steps, warmup)
            del g2
    group = 8
    multi_us = None
    if w.steps % group == 0 and args.steps >= group:
        g8 = capture(args.step, group)
        multi_us = replay_pass(args.step, g8, max(1, args.steps // group), max(1, warmup // group), group)
        del g8
    # what the apply kernel adds to a replayed three-launch step (launch overlap and kernel boundary included)
    t_apply_in_step = max(by_mode["three"] - by_mode["no_apply"], 1e-3)

    # ---- pass B: per-kernel device times over the same steps -----------------------------------
    # Eager calls with events between them.  A short spin kernel in front of every step lets the
    # host queue the whole step before the GPU starts it, so the event intervals are device time
    # (kernel + launch gap) rather than host issue time.
    restart("three")
    spin_cycles = int(2.0e5)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    zero_bits_sum, mask_samples = 0, 0
    sector_stats = np.zeros(3)
    fill_work = {"merge_bytes": 0, "check_bytes": 0, "row_bytes": 0, "check_tokens": 0, "steps": 0}
    for i in range(total):
        t = i % w.steps
        if t == 0 and i > 0:
            restart("three")
        buf = ring[i % ring_n]
        ev = evs[i - warmup] if i >= warmup else None
        torch.cuda._sleep(spin_cycles)
        if ev:
            ev[0].record()
        s.fill()
        if ev:
            ev[1].record()
        s.apply(buf)
        if ev:
            ev[2].record()
        s.accept_device(traj[t], restart_on_eos=True)
        if ev:
            ev[3].record()
        if ev and (i - warmup) % 10 == 0:            # masked fraction, sampled (synchronises; outside the event intervals)
            bits = np.unpackbits(s.mask_numpy().view(np.uint8), axis=1, bitorder="little")[:, :s.V]
            zero_bits_sum += n * s.V - int(bits.sum())
            mask_samples += 1
            # the 32-byte sectors of the logits by what the mask does to them: untouched, overwritten, read and rewritten
            per_sector = 32 // elt
            sec = bits[:, :s.V // per_sector * per_sector].reshape(n, -1, per_sector).sum(axis=2)
            sector_stats += [int((sec == per_sector).sum()), int((sec == 0).sum()), int(((sec > 0) & (sec < per_sector)).sum())]
            for m in s.matchers:                       # what the next fill streams: cache entries merged, candidates tested, row written
                fw = m.next_fill_work(s.stream())
                fill_work["merge_bytes"] += fw["merge_bytes"]; fill_work["check_bytes"] += fw["check_bytes"]
                fill_work["row_bytes"] += fw["row_bytes"]; fill_work["check_tokens"] += fw["check_tokens"]
            fill_work["steps"] += 1
    torch.cuda.synchronize()
    eager_us = {"fill": float(np.mean([e[0].elapsed_time(e[1]) for e in evs])) * 1e3,
                "apply": float(np.mean([e[1].elapsed_time(e[2]) for e in evs])) * 1e3,
                "accept": float(np.mean([e[2].elapsed_time(e[3]) for e in evs])) * 1e3}

    # the two-in-one launches, timed the same way
    for name, mode in (("accept_fill", "accept_fill"), ("fill_apply", "fill_apply")):
        restart(mode)
        evf = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        for i in range(total):
            t = i % w.steps
            if t == 0 and i > 0:
                restart(mode)
            ev = evf[i - warmup] if i >= warmup else None
            torch.cuda._sleep(spin_cycles)
            if mode == "accept_fill":
                s.apply(ring[i % ring_n])
            if ev:
                ev[0].record()
            if mode == "accept_fill":
                s.accept_fill_device(traj[t], restart_on_eos=True)
            else:
                s.fill_apply(ring[i % ring_n])
            if ev:
                ev[1].record()
            if mode == "fill_apply":
                s.accept_device(traj[t], restart_on_eos=True)
        torch.cuda.synchronize()
        eager_us[name] = float(np.mean([e[0].elapsed_time(e[1]) for e in evf])) * 1e3

    # ---- apply alone: launches back to back over the logits ring (the last step's mask) ---------
    # The intervals above hold the launch gap of a short kernel; a stream of launches does not.
    reps = 4 * ring_n
    for k in range(ring_n):
        s.apply(ring[k])
    torch.cuda.synchronize()
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(int(4.0e6))       # about 2 ms: the host queues every launch below before the GPU starts the first
    a0.record()
    for k in range(reps):
        s.apply(ring[k % ring_n])
    a1.record()
    torch.cuda.synchronize()
    t_apply_alone = a0.elapsed_time(a1) * 1e3 / reps
    alone_zero_bits = n * s.V - int(np.unpackbits(s.mask_numpy().view(np.uint8)).sum())
    # the same launches with a mask that allows nothing: every vector is overwritten and none is read, i.e. what the
    # memory system takes from this kernel as a pure store stream of the same size (the mask is still read first)
    saved_mask = s.bitmask.clone()
    s.bitmask.zero_()
    for k in range(ring_n):
        s.apply(ring[k])
    torch.cuda.synchronize()
    torch.cuda._sleep(int(4.0e6))
    a0.record()
    for k in range(reps):
        s.apply(ring[k % ring_n])
    a1.record()
    torch.cuda.synchronize()
    t_apply_all_masked = a0.elapsed_time(a1) * 1e3 / reps
    s.bitmask.copy_(saved_mask)
    del saved_mask
    clocks = sampler.finish()          # sampled over the timed pass and the per-kernel passes (same steps, same kernels)
    t_fill, t_apply, t_accept = eager_us["fill"], eager_us["apply"], eager_us["accept"]
    zero_bits = zero_bits_sum / max(mask_samples, 1)

    # apply's algorithmic bytes: the mask words read plus the masked logits written (allowed
    # logits are neither read nor written); and the conventional count (read + write everything)
    masked_frac = zero_bits / float(n * s.V)
    apply_alg_bytes = 4.0 * n * W + elt * zero_bits
    apply_conv_bytes = 2.0 * elt * n * s.V + 4.0 * n * W
    # what has to cross the memory interface in 32-byte sectors: the mask, every sector with a masked logit written,
    # every sector that mixes allowed and masked logits read first
    sec_untouched, sec_overwritten, sec_mixed = (sector_stats / max(mask_samples, 1)).tolist()
    apply_sector_bytes = 4.0 * n * W + 32.0 * (sec_overwritten + 2 * sec_mixed)
    peak, peak_kind = measured_peaks()
    ncu = ncu_figures(args.workload, n)
    traffic = ncu.get("apply_kernel", {}).get("dram_bytes")          # ncu: DRAM bytes read + written per launch; None once the kernels changed
    apply_gbs = apply_alg_bytes / (t_apply_in_step * 1e-6) / 1e9
    dominant = max((("fill", t_fill), ("apply", t_apply), ("accept", t_accept)), key=lambda x: x[1])[0]

    def apply_at(t_us, zb=None):
        alg = apply_alg_bytes if zb is None else 4.0 * n * W + elt * zb
        return {"us_per_launch": t_us, "achieved": alg / (t_us * 1e-6) / 1e9, "frac": alg / (t_us * 1e-6) / 1e9 / peak,
                "sector_traffic_gbs": apply_sector_bytes / (t_us * 1e-6) / 1e9, "sector_traffic_frac": apply_sector_bytes / (t_us * 1e-6) / 1e9 / peak,
                "ncu_traffic_frac": (traffic / (t_us * 1e-6) / 1e9 / peak) if traffic else None,
                "conventional_gbs": apply_conv_bytes / (t_us * 1e-6) / 1e9}

    roofline = {"kernel": "apply_kernel", "bound": "hbm", "achieved": apply_gbs, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": apply_gbs / peak, "traffic": traffic, "us_per_launch": t_apply_in_step,
                "how": "in-graph: replayed three-launch step (fill, apply, accept) minus the same step without its apply",
                "masked_fraction": masked_frac, "algorithmic_bytes": apply_alg_bytes,
                "sector_bytes": apply_sector_bytes, "sectors": {"untouched": sec_untouched, "overwritten": sec_overwritten, "read_and_rewritten": sec_mixed},
                "in_step": apply_at(t_apply_in_step), "dominant_by_time": dominant,
                "eager_event_interval": apply_at(t_apply),
                "alone": dict(apply_at(t_apply_alone, alone_zero_bits),
                              how="%d launches back to back over the logits ring (queued behind a primer kernel), last step's mask" % reps),
                "alone_all_masked": dict({k_: v_ for k_, v_ in apply_at(t_apply_all_masked, n * s.V).items() if k_ in ("us_per_launch", "achieved", "frac")},
                                         how="the same launches with an all-zero mask: stores only, no logit is read (the store ceiling of this kernel and size)")}

    # The fill and accept kernels are bound by latency, not by a memory or arithmetic pipe.  What can be said against a
    # peak is their issue rate: warp instructions per launch (ncu) over the launch time, against 148 SMs x 4 schedulers
    # x the SM clock.
    props = torch.cuda.get_device_properties(local_rank)
    issue_peak = props.multi_processor_count * 4 * (clocks["sm_max_mhz"] or 1965.0) * 1e6
    latency_bound = {}
    for name, kernel, t_us in (("fill", "fill_cluster_kernel", t_fill), ("accept", "accept_kernel", t_accept)):
        wi = ncu.get(kernel, {}).get("warp_instructions")
        latency_bound[name] = {"kernel": kernel, "bound": "alu",
                               "achieved": (wi / (t_us * 1e-6)) if wi else None, "peak": issue_peak, "unit": "warp instructions/s",
                               "frac": (wi / (t_us * 1e-6) / issue_peak) if wi else None, "warp_instructions_per_launch": wi,
                               "us_per_launch": t_us, "note": "latency-bound: chains of dependent loads"}

    fw_steps = max(fill_work["steps"], 1)
    fill_bytes = (fill_work["merge_bytes"] + fill_work["check_bytes"] + fill_work["row_bytes"]) / fw_steps
    fill_stream = {"bytes_per_launch": fill_bytes, "merge_bytes": fill_work["merge_bytes"] / fw_steps, "check_bytes": fill_work["check_bytes"] / fw_steps,
                   "row_bytes": fill_work["row_bytes"] / fw_steps, "uncertain_candidates_per_launch": fill_work["check_tokens"] / fw_steps,
                   "gbs": fill_bytes / (t_fill * 1e-6) / 1e9, "frac_of_hbm_peak": fill_bytes / (t_fill * 1e-6) / 1e9 / peak,
                   "sampled_steps": fill_work["steps"]}
    t_fa = eager_us["fill_apply"]
    fused = {"kernel": "fill_cluster_kernel with the apply tail", "us_per_launch": t_fa, "us_fill_then_apply_as_two_launches": t_fill + t_apply,
             "algorithmic_bytes": apply_alg_bytes - 4.0 * n * W + fill_bytes,
             "achieved_gbs": (apply_alg_bytes - 4.0 * n * W + fill_bytes) / (t_fa * 1e-6) / 1e9,
             "frac_of_hbm_peak": (apply_alg_bytes - 4.0 * n * W + fill_bytes) / (t_fa * 1e-6) / 1e9 / peak,
             "note": "the launch lasts as long as its slowest request's token walks; the logits traffic of the other rows overlaps them"}

    # ---- end to end through the C ABI with host buffers ---------------------------------------
    # Every step: the step's logits come from pinned host memory, the masked logits go back to pinned host memory,
    # the step's token ids come from the host.  Two device buffers and two copy streams, as a serving loop would
    # have them: the upload of step t+1 and the download of step t-1 overlap the kernels of step t (PCIe is full
    # duplex); every dependency is an event, nothing is skipped.
    e2e_mode = args.step if args.step != "no_apply" else "fill_apply"
    e2e_steps = max(4, min(args.steps, 16))
    host_in = torch.empty((n, s.V), dtype=tdtype).pin_memory()
    host_in.copy_(ring[0].cpu())
    host_out = [torch.empty((n, s.V), dtype=tdtype).pin_memory() for _ in range(2)]
    host_traj = traj.cpu().pin_memory()
    dev_buf = [ring[0], ring[1 % ring_n]]
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for phase in ("warm", "timed"):
        restart(e2e_mode)
        torch.cuda.synchronize()
        if phase == "timed":
            h0.record()
        ev_in = [None, None]
        ev_out = [None, None]
        ev_applied = [None, None]

        def upload(t):
            k = t % 2
            with torch.cuda.stream(s_in):
                if ev_out[k] is not None:
                    s_in.wait_event(ev_out[k])          # the buffer's previous contents have left the device
                dev_buf[k].copy_(host_in, non_blocking=True)
                ev_in[k] = torch.cuda.Event()
                ev_in[k].record(s_in)

        if phase == "timed":
            s_in.wait_event(h0)
        upload(0)
        for t in range(e2e_steps):
            k = t % 2
            if t + 1 < e2e_steps:
                upload(t + 1)
            if e2e_mode == "three":
                s.fill()
            main.wait_event(ev_in[k])
            if e2e_mode == "fill_apply":
                s.fill_apply(dev_buf[k])
            else:
                s.apply(dev_buf[k])
            ev_applied[k] = torch.cuda.Event()
            ev_applied[k].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_applied[k])
                host_out[k].copy_(dev_buf[k], non_blocking=True)
                ev_out[k] = torch.cuda.Event()
                ev_out[k].record(s_out)
            s.tokens.copy_(host_traj[t], non_blocking=True)
            if e2e_mode == "accept_fill":
                s.accept_fill_device(s.tokens, restart_on_eos=True)
            else:
                s.accept_device(s.tokens, restart_on_eos=True)
        main.wait_event(ev_out[0])
        main.wait_event(ev_out[1])
        if phase == "timed":
            h1.record()
        torch.cuda.synchronize()
    e2e_us = dist_util.max_over_ranks(h0.elapsed_time(h1)) * 1e3 / e2e_steps

    launch_text = {"fill_apply": "fill + apply in one launch, then accept", "three": "fill, apply, accept",
                   "accept_fill": "apply, then accept + fill of the next mask in one launch"}[args.step]
    classify_ms = sum(x["classify_ms"] for x in stats)
    # the work behind a classified pair: token bytes the walks consume (viable trie nodes, no sharing between tokens),
    # counted in a second compile of the first grammars into a pool of their own (the timed compile does not count)
    cpool = XB.CachePool(s.tokenizer)
    counted = [XB.Grammar(s.tokenizer, g.kind, g.text, pool=cpool, count_node_visits=True) for g in w.grammars[:16]]
    cstats = [g.stats() for g in counted]
    visits_per_pair = sum(x["node_visits"] for x in cstats) / max(sum(x["pairs_classified"] for x in cstats), 1)
    for g in counted:
        g.close()
    cpool.close()
    line = {
        "metric": metric, "value": us_per_step, "unit": "us/step", "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": us_per_step / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32", "data": "synthetic",
        "config": {"workload": args.workload, "batch": n, "global_batch": n * world, "vocab": s.V, "logits_dtype": w.dtype, "launch": "one CUDA graph per trajectory step: " + launch_text,
                   "grammars": len(w.grammars), "l2": "logits ring of %d buffers (%.0f MB) > 2 x L2" % (ring_n, ring_n * bytes_one / 1e6),
                   "parallelism": "replicas x%d" % world},
        "clocks": clocks,
        "us_per_step_by_launch_structure": by_mode,
        "us_per_step_with_8_steps_per_graph": multi_us,
        "kernels_us": {"fill": t_fill, "apply": t_apply, "accept": t_accept, "accept_fill": eager_us["accept_fill"], "fill_apply": eager_us["fill_apply"],
                       "apply_in_step": t_apply_in_step},
        "apply_gbs": apply_gbs,
        "cache_build": {"seconds": build_ms / 1e3, "compile_wall_s": compile_s, "session_wall_s": session_s, "compile_threads": args.compile_threads or min(16, os.cpu_count() or 1), "pairs_classified": pairs, "pairs_per_s": pairs / max(build_ms / 1e3, 1e-9),
                        "pairs_per_s_of_wall_time": pairs / max(compile_s, 1e-9),
                        "pairs_dense": pairs_dense, "pairs_dense_per_s": pairs_dense / max(build_ms / 1e3, 1e-9),
                        "classify_kernel_ms": classify_ms,
                        "pairs_per_s_classify_kernel": pairs / max(classify_ms / 1e3, 1e-9),
                        "viable_node_visits_per_pair": visits_per_pair,
                        "viable_node_visits_per_s": visits_per_pair * pairs / max(classify_ms / 1e3, 1e-9),
                        "entries_built": sum(x["n_entries_built"] for x in stats), "entries_reused": sum(x["n_entries_reused"] for x in stats),
                        "entries_shared_by_state_compression": sum(x["n_entries_shared"] for x in stats), "states": sum(x["n_states"] for x in stats),
                        "frontend_ms": sum(x["frontend_ms"] for x in stats),
                        "uncertain_total": sum(x["total_uncertain"] for x in stats), "uncertain_after_lookahead": sum(x["total_checked"] for x in stats),
                        "cache_bytes_unique_upper": sum(x["cache_bytes"] for x in stats)},
        "roofline": roofline,
        "roofline_latency_bound_kernels": latency_bound,
        "fill_streaming": fill_stream,
        "fill_and_apply_in_one_launch": fused,
        "e2e": {"value": e2e_us, "unit": "us/step", "h2d_bytes_per_step": bytes_one + 4 * n, "d2h_bytes_per_step": bytes_one, "steps": e2e_steps},
        "gpu_launches": timed_launches,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        us, threads, sample = oracle_leg(w, args.steps, args.warmup)
        us1, _, sample1 = oracle_leg(w, args.steps, args.warmup, threads=1, n_req=4, budget_s=12.0)
        n_built = sum(x["n_entries_built"] for x in stats)
        line["cpu_baseline"] = {"value": us, "unit": "us/step", "cores": threads, "kind": "oracle", "sample": sample,
                                "single_thread": {"value": us1, "unit": "us/step", "us_per_mask": us1 / n, "sample": sample1},
                                "cache_build": {"all_cores": oracle_cache_build_leg(w, n_built, threads), "single_thread": oracle_cache_build_leg(w, n_built, 1, n_positions=12, budget_s=6.0)}}
    s.close()
    # the same compile into a pool whose device memory was taken from the driver beforehand (a server that reserves its
    # cache budget at start-up): what is left is the build itself
    s2 = engine.Session(w, device="cuda:%d" % local_rank, state_compression=not args.no_state_compression, compile_threads=args.compile_threads,
                        reserve_bytes=int(pool_reserved * 1.25) + (64 << 20), repeat_threshold=args.repeat_threshold)
    st2 = [g.stats() for g in s2.grammars]
    line["cache_build"]["with_reserved_pool"] = {"seconds": sum(x["cache_build_ms"] for x in st2) / 1e3, "compile_wall_s": s2.compile_wall_s,
                                                 "pairs_per_s": pairs / max(sum(x["cache_build_ms"] for x in st2) / 1e3, 1e-9),
                                                 "pairs_per_s_of_wall_time": pairs / max(s2.compile_wall_s, 1e-9), "reserved_bytes": int(pool_reserved * 1.25) + (64 << 20)}
    s2.close()
    if rank == 0:
        print(json.dumps(line))
    dist_util.finish()
    return 0


def jit_sweep(w, args, local_rank):
    """Per-step time with the cache built just in time (Section 3.5): for each K, compile with K entries
    precomputed, then run the trajectory once from a cold pool (entries arrive while decoding) and once more
    warm.  A step = fill + apply + accept + the service call and whatever cache-build kernels it enqueued."""
    import torch
    from paper_2601_04426_b200 import binding as XB
    from paper_2601_04426_b200 import engine
    wt = XB.Tokenizer([bytes([i]) for i in range(256)] + [b""], 256, [])
    XB.Grammar(wt, "ebnf", 'root ::= [a-z]+ "."').close()
    wt.close()
    rows = []
    n = w.batch
    for k_text in args.jit_sweep.split(","):
        full = k_text == "full"
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        s = engine.Session(w, device="cuda:%d" % local_rank, jit=not full, jit_precompute=0 if full else int(k_text))
        torch.cuda.synchronize()
        compile_s = time.perf_counter() - t0
        stats = [g.stats() for g in s.grammars]
        logits = engine.logits_tensor(inputs.make_logits(w.logits_seed, min(n, 8), s.V, w.dtype), s.device)
        logits = logits.repeat((n + logits.shape[0] - 1) // logits.shape[0], 1)[:n].contiguous()
        traj = torch.from_numpy(np.asarray([[w.trajectories[b][t] for b in range(n)] for t in range(w.steps)], dtype=np.int32)).to(s.device)
        eos_at = {t: [b for b in range(n) if w.trajectories[b][t] == w.vocab.eos_id] for t in range(w.steps)}
        passes = {}
        for label in ("cold", "warm"):
            if label == "warm" and not full:
                s.jit_service(wait=True)          # whatever the cold pass left in flight or unreported
            for b in range(n):
                s.reset(b)
            torch.cuda.synchronize()
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(w.steps + 1)]
            evs[0].record()
            for t in range(w.steps):
                s.fill()
                s.apply(logits)
                s.accept_device(traj[t])
                for b in eos_at[t]:
                    s.reset(b)
                if not full:
                    s.jit_service(wait=False)
                evs[t + 1].record()
                evs[t + 1].synchronize()        # a decode loop waits here for the sampled tokens: the host never runs ahead of the GPU
            torch.cuda.synchronize()
            us = np.asarray([evs[t].elapsed_time(evs[t + 1]) * 1e3 for t in range(w.steps)])
            passes[label] = {"avg_us": float(us.mean()), "p99_us": float(np.percentile(us, 99)), "max_us": float(us.max())}
        js = s.jit_service(wait=True) if not full else {"n_built": 0, "n_pool_hits": 0, "n_missing": 0}
        rows.append({"K": k_text, "compile_wall_s": compile_s, "cache_build_ms": sum(x["cache_build_ms"] for x in stats),
                     "frontend_ms": sum(x["frontend_ms"] for x in stats),
                     "entries_built_at_compile": sum(x["n_entries_built"] for x in stats), "entries_built_just_in_time": js["n_built"],
                     "pool_hits": js["n_pool_hits"], "entries_never_built": js["n_missing"], "steps": w.steps, **{k + "_" + kk: vv for k, p in passes.items() for kk, vv in p.items()}})
        s.close()
    return {"metric": "per-step us with just-in-time cache build (eager launches: fill, apply, accept, service)", "workload": w.name, "batch": n,
            "vocab": w.vocab.size, "rows": rows}


def _with_batch(w, batch):
    """A workload whose nominal batch is `batch` while only the first requests are materialised."""
    class _View:
        pass
    v = _View()
    v.__dict__.update(w.__dict__)
    v.batch = batch
    return v


if __name__ == "__main__":
    sys.exit(main())
