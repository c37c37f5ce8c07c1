#!/usr/bin/env python
"""Benchmark of the first-layer cached attention path (RoPECache + FACache).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload CFG] [--impl reference]

A "step" is one denoising step of the block schedule: `lacache_step` (RoPE-on-
write of the block, fixed queries x block keys merged with the cached state,
block queries x all keys); the first step of every block is preceded by that
block's `lacache_build`, which is inside the timed region.  The headline value
is denoising steps/s over K calls issued back to back on several replicas of
the cache state visited round-robin, so that every call finds its inputs in
HBM rather than in L2 (inputs larger than L2; in a real model 31 other layers
run between two calls of this one).  Beside it: the old per-call figure with a
flushed L2, a warm-L2 figure from one CUDA-graph replay on one replica, and
`e2e`, the same schedule through the host-buffer entry points.

With N > 1 (one process per GPU under torchrun) every rank runs its own seeded
batch of the same workload: the path has no exchange step, so there is no
collective on the data path; only the timing is reduced (max over ranks).

`--impl reference` times the fp64 CPU oracle (the only reference there is for
this path) on the host cores instead.
"""
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

METRIC = "layer-1 denoising steps/s (LLaDA-8B shape, cached first-layer attention)"
UNIT = "steps/s"


# ----------------------------------------------------------------------------
# workload arithmetic (counts only)
# ----------------------------------------------------------------------------
def flops_and_bytes(wl):
    """Algorithmic work of one step / one build, summed over the batch.

    Flops: 4 d Hq [(N - Lb) Lb + Lb N] per step, 4 d Hq (N - Lb)^2 per build.
    Bytes of the step attention kernel: rotated Q of fixed rows (2 B/el), cached
    O~ (4 B/el) and m, l (8 B/row-head), all rotated K and V (2 B/el), rotated Q
    of block rows, and the fp32 output of all rows.  Bytes of the whole step add
    the block's pre-RoPE read and rotated write.  Extra planes the
    implementation keeps for precision (the lo halves of Q and K) are overhead,
    not algorithmic bytes.
    """
    d, Hq, Hkv, Lb = wl.head_dim, wl.n_q_heads, wl.n_kv_heads, wl.block_len
    e = 2 if wl.dtype == "bf16" else 4
    step_flops = build_flops = 0
    attn_bytes = rope_bytes = build_bytes = 0
    for N in wl.seq_lens:
        step_flops += 4 * d * Hq * ((N - Lb) * Lb + Lb * N)
        build_flops += 4 * d * Hq * (N - Lb) ** 2
        attn_bytes += (N - Lb) * Hq * (d * (e + 4) + 8) + 2 * N * Hkv * d * e + Lb * Hq * d * e + N * Hq * d * 4
        rope_bytes += 2 * Lb * (Hq + 2 * Hkv) * d * e
        build_bytes += 2 * N * (Hq + 2 * Hkv) * d * e + (N - Lb) * Hq * (d * 4 + 8) + \
            (N - Lb) * Hq * d * e + 2 * N * Hkv * d * e
    return dict(step_flops=step_flops, build_flops=build_flops, step_attn_bytes=attn_bytes,
                step_bytes=attn_bytes + rope_bytes, build_bytes=build_bytes)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm_gbs=j["hbm_gbs"], bf16_tflops=j["bf16_tflops"],
                    bf16_tflops_sustained=j["bf16_tflops_sustained"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------
# clocks sampler
# ----------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.samples = []
        self.window = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "5"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.perf_counter(), line.strip()))

    def mark(self):
        """Start (first call) / end (second call) of the window whose samples count."""
        self.window.append(time.perf_counter())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        lo, hi = (self.window + [None, None])[:2]
        inside = [l for t, l in self.samples if (lo is None or t >= lo) and (hi is None or t <= hi + 0.01)]
        if len(inside) < 3:      # a very short window: fall back to every sample taken
            inside = [l for _, l in self.samples]
        for s in inside:
            f = [x.strip() for x in s.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx = float(f[1])
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------
# distributed plumbing (timing only; the data path has no exchange)
# ----------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def reduce_max(value, backend_device="cuda"):
    """Max of a python float over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=backend_device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def rank_seed(base_seed, rank):
    """Each rank draws its own batch: same shapes, different seeded values."""
    return base_seed * 1000003 + rank


# ----------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------
L2_BYTES = 126 << 20


def n_replicas(step_bytes):
    """Cache states visited round-robin so that a state's lines have left the L2
    before it is touched again: the other replicas' steps move at least twice
    the L2 capacity in between."""
    import math
    if step_bytes >= 8 * L2_BYTES:      # one step alone moves many times the L2
        return 1
    return max(3, math.ceil(2.0 * L2_BYTES / max(step_bytes, 1)) + 1)


def replica_phases(K, R, S):
    """Step-in-block index of every replica's first timed call, chosen so that K calls visiting the R
    replicas round-robin contain round(K / S) builds (at least one once K >= 8): a build falls due when a
    replica reaches step 0 of a block.  Returns (phases, builds the K calls will contain)."""
    n = [(K - c + R - 1) // R if c < K else 0 for c in range(R)]
    builds = lambda p, m: sum(1 for q in range(m) if (p + q) % S == 0)
    target = round(K / S)
    if K >= 8:
        target = max(1, target)
    base = sum(m // S for m in n)
    cand = [c for c in range(R) if n[c] > 0 and n[c] % S != 0]
    extra = max(0, min(len(cand), target - base))
    chosen = set(cand[int((j + 0.5) * len(cand) / extra)] for j in range(extra)) if extra else set()
    phases = []
    for c in range(R):
        m = n[c]
        want = m // S + (1 if c in chosen else 0)
        if m >= S:
            pref = (c * max(1, S // R)) % S              # long runs: block boundaries staggered over the replicas
        else:
            pref = (S - m // 2) % S if c in chosen else 1  # the one build in the middle of the replica's calls
        ok = [p for p in range(S) if builds(p, m) == want] or list(range(S))
        phases.append(min(ok, key=lambda p: min((p - pref) % S, (pref - p) % S)))
    return phases, sum(builds(p, m) for p, m in zip(phases, n))


class RoundRobin:
    """K calls over R cache states visited round-robin, every replica walking its own block schedule:
    a step per call, preceded by the block's build whenever the replica enters a new block."""

    def __init__(self, ctxs, outs, sched, K, S):
        self.ctxs, self.outs, self.sched, self.K, self.S = ctxs, outs, sched, K, S
        self.R = len(ctxs)
        self.phases, self.n_builds = replica_phases(K, self.R, S)
        self.total = sched.n_blocks_used * S
        self.local = [0] * self.R

    def prepare(self):
        """Untimed: every replica gets the cache of the block in which the step BEFORE its first timed call
        lies, and runs that step (so each replica has stepped at least once, and a replica whose phase is 0
        meets its build inside the timed region)."""
        for c in range(self.R):
            first = ((c % self.sched.n_blocks_used) * self.S + self.phases[c]) % self.total
            prev = (first - 1) % self.total
            blk, _, tens = self.sched.step_inputs(prev)
            self.ctxs[c].build(blk, *self.sched.full[blk])
            self.ctxs[c].step(*tens, *self.outs[c])
            self.local[c] = first

    def run(self, n_calls=None, on_call=None, stream=None):
        """The calls themselves (on `stream`, default the current one).  Returns (kernel launches, builds)."""
        kw = {} if stream is None else {"stream": stream}
        launches = builds = 0
        for j in range(self.K if n_calls is None else n_calls):
            c = j % self.R
            blk, s, tens = self.sched.step_inputs(self.local[c])
            ctx = self.ctxs[c]
            if s == 0:
                if on_call:
                    on_call("build", ctx)
                ctx.build(blk, *self.sched.full[blk], **kw)
                launches += ctx.last_launch_count
                builds += 1
                if on_call:
                    on_call("built", ctx)
            if on_call:
                on_call("step", ctx)
            ctx.step(*tens, *self.outs[c], **kw)
            launches += ctx.last_launch_count
            if on_call:
                on_call("stepped", ctx)
            self.local[c] = (self.local[c] + 1) % self.total
        return launches, builds


def timed_region(rr, W, min_ms=50.0, max_repeats=200, graph=True):
    """W untimed warm-up calls, then the K-call region `repeats` times, each bracketed by one event pair
    (barrier + synchronize on both sides) after an untimed pass that puts every replica at its phase.
    With `graph` the K calls (the library's own launches, in the same order, programmatic dependencies
    included) are captured once into a CUDA graph and every repeat replays it: the host's time to enqueue
    two launches per step through Python is of the order of the step itself, and a denoising loop that
    cares captures its step the same way.  rr.launch says which of the two ran.
    Returns (per-repeat ms, launches per repeat, builds per repeat, wall seconds of the timed regions)."""
    import math
    import torch
    mk = lambda: torch.cuda.Event(enable_timing=True)
    rr.prepare()
    rr.run(W)
    torch.cuda.synchronize()
    g = gs = None
    launches = builds = 0
    if graph:
        try:
            gs = torch.cuda.Stream()
            rr.prepare()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(gs):
                with torch.cuda.graph(g, stream=gs):
                    launches, builds = rr.run(stream=gs.cuda_stream)
            torch.cuda.synchronize()
        except Exception as ex:      # (capture is a convenience of the harness: without it the calls are issued one by one)
            sys.stderr.write("graph capture of the timed region skipped: %r\n" % (ex,))
            g = None
    rr.launch = "cuda graph replay" if g is not None else "eager"
    times, wall = [], 0.0
    repeats = 1
    i = 0
    while i < repeats:
        rr.prepare()
        torch.cuda.synchronize(); barrier()
        t0 = time.perf_counter()
        e0, e1 = mk(), mk()
        if g is not None:
            with torch.cuda.stream(gs):
                e0.record()
                g.replay()
                e1.record()
        else:
            e0.record()
            launches, builds = rr.run()
            e1.record()
        torch.cuda.synchronize(); barrier()
        wall += time.perf_counter() - t0
        times.append(e0.elapsed_time(e1))
        if i == 0:   # size the number of repeats from the first one (the same on every rank: max over ranks)
            t1 = reduce_max(times[0], torch.device("cuda", torch.cuda.current_device()))
            repeats = 1 if t1 >= 4 * min_ms else max(5, min(max_repeats, math.ceil(min_ms / max(t1, 1e-3))))
        i += 1
    return times, launches, builds, wall


def run_cuda(args):
    import torch
    from paper_2607_16339_b200 import binding
    from paper_2607_16339_b200.workloads import WORKLOADS, DeviceSchedule

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    wl = WORKLOADS[args.workload]
    K, W = args.steps, args.warmup
    S = wl.steps_per_block
    counts = flops_and_bytes(wl)
    peaks = load_peaks()
    T = wl.total_tokens
    mk = lambda: torch.cuda.Event(enable_timing=True)
    # (default: one fp16 plane per operand where the workload's full-size parity test passes with it --
    # tests/test_gpu_parity.py::test_full_size_configs_at_parity_points and the large-batch test -- the
    # split bf16 planes for the workload whose keys carry 4x outliers; the split figure is reported beside)
    precision = DEFAULT_PRECISION.get(wl.cfg, binding.PRECISION_SPLIT) if args.precision_mode < 0 else args.precision_mode
    out_bf16 = args.out_dtype == "bf16"
    ctx_kw = dict(precision_mode=precision, out_dtype=binding.OUT_BF16 if out_bf16 else binding.OUT_FP32)
    out_t = torch.bfloat16 if out_bf16 else torch.float32

    # ---- replicas: independent cache states of the same workload, visited round-robin ----
    # Every call then finds its inputs (cached state, rotated planes) in HBM, not in L2,
    # while the calls run back to back as they do in a denoising loop.
    R = args.replicas or n_replicas(counts["step_attn_bytes"])
    sched = DeviceSchedule(wl, rank_seed(args.seed, rank), dev, min(wl.n_steps, 3 * S))

    def make_replicas(**kw):
        cs = [binding.Context.from_workload(wl, **dict(ctx_kw, **kw)) for _ in range(R)]
        for c in cs:
            c.set_step_overlap(True)     # the step inputs are all resident before the first call
        return cs

    ctxs = make_replicas()
    outs = [(torch.empty(T, wl.n_q_heads, wl.head_dim, device=dev, dtype=out_t), torch.empty(T, wl.n_q_heads, device=dev))
            for _ in range(R)]
    ctx = ctxs[0]
    tc = ctx.engine == binding.ENGINE_TCGEN05

    clocks = ClockSampler(local_rank)
    clocks.start()
    time.sleep(0.05)   # let the sampler come up
    # ---- headline: K calls back to back, builds pro rata, one event pair around each repeat ----
    rr = RoundRobin(ctxs, outs, sched, K, S)
    clocks.mark()
    times, launches, n_builds, t_wall = timed_region(rr, W)
    total_ms = statistics.median(times)
    launch_mode = rr.launch
    eager_ms = None
    if launch_mode != "eager":      # the same calls issued one by one from Python, for comparison
        etimes, _, _, _ = timed_region(rr, 3, min_ms=20.0, graph=False)
        eager_ms = statistics.median(etimes)

    # ---- per-kernel durations of the attention kernels: the same calls again, with an event
    # pair recorded inside the library around each attention kernel (no host sync in between) ----
    events = []

    def with_events(kind, c):
        if kind in ("build", "step"):
            e = (mk(), mk()); e[0].record(); e[1].record()
            c.set_timing_events(*e); events.append((kind, e))

    rrk = RoundRobin(ctxs, outs, sched, max(min(K, 256), S * R // 4), S)
    rrk.prepare()
    rrk.run(on_call=with_events)
    torch.cuda.synchronize()
    for c in ctxs:
        c.set_timing_events(None, None)
    kern_step_ms = [a.elapsed_time(b) for kind, (a, b) in events if kind == "step"]
    kern_build_ms = [a.elapsed_time(b) for kind, (a, b) in events if kind == "build"]
    if not kern_build_ms:     # no block boundary in the range: time one build on its own
        e = (mk(), mk()); e[0].record(); e[1].record()
        ctx.set_timing_events(*e)
        ctx.build(0, *sched.full[0]); torch.cuda.synchronize()
        ctx.set_timing_events(None, None)
        kern_build_ms.append(e[0].elapsed_time(e[1]))

    # ---- the same calls once more, back to back and overlapping as in the headline, with every launch of
    # the attention kernel stamping the GPU's global timer at its first CTA's entry and last CTA's exit ----
    span = None
    if tc:
        n_slots = 16 * (rrk.K // R + 2) + 8
        rings = [torch.empty(n_slots, 2, dtype=torch.int64, device=dev) for _ in range(R)]
        for r_ in rings:
            r_[:, 0] = -1       # UINT64_MAX
            r_[:, 1] = 0
        kinds = [[] for _ in range(R)]
        idx = {id(c): i for i, c in enumerate(ctxs)}

        def note(kind, c):
            if kind in ("built", "stepped"):
                kinds[idx[id(c)]].append((kind, c.last_launch_count - 1))     # (one RoPE launch per call)

        rrk.prepare()
        torch.cuda.synchronize()
        for c, r_ in zip(ctxs, rings):
            c.set_span_ring(r_)
        rrk.run(on_call=note)
        torch.cuda.synchronize()
        for c in ctxs:
            c.set_span_ring(None)
        sp = {"stepped": [], "built": []}
        for r_, ks in zip(rings, kinds):
            h = r_.cpu().numpy()
            slot = 0
            for kind, n in ks:       # a call's launches (several when a step's fixed rows go out in more than one)
                if slot + n > n_slots:
                    break
                if n > 0:
                    sp[kind].append(float(h[slot:slot + n, 1].max() - h[slot:slot + n, 0].min()) * 1e-3)     # ns -> us
                slot += n
        if sp["stepped"]:
            span = {"step_us": round(statistics.mean(sp["stepped"]), 2),
                    "step_us_median": round(statistics.median(sp["stepped"]), 2),
                    "build_us": round(statistics.mean(sp["built"]), 2) if sp["built"] else None,
                    "launches": len(sp["stepped"]),
                    "how": "first CTA entry to last CTA exit of the attention kernel's launches (global timer, "
                           "stamped by the kernel), calls back to back and overlapping as in the headline"}

    # ---- GPU full recompute of the same step (the vanilla pass the method replaces), same round-robin ----
    n_fr = max(2 * R, 16)
    fulls = [sched.full[c % sched.n_blocks_used] for c in range(R)]
    for c in range(R):
        ctxs[c].full_recompute(*fulls[c], *outs[c])
    torch.cuda.synchronize(); barrier()
    e0, e1 = mk(), mk()
    e0.record()
    for i in range(n_fr):
        ctxs[i % R].full_recompute(*fulls[i % R], *outs[i % R])
    e1.record()
    torch.cuda.synchronize()
    fr_ms = e0.elapsed_time(e1) / n_fr
    fr_pairs = []
    for i in range(min(n_fr, 16)):
        e = (mk(), mk()); e[0].record(); e[1].record()
        ctxs[i % R].set_timing_events(*e); fr_pairs.append(e)
        ctxs[i % R].full_recompute(*fulls[i % R], *outs[i % R])
    torch.cuda.synchronize()
    for c in ctxs:
        c.set_timing_events(None, None)
    fr_kernel_ms = statistics.mean(a.elapsed_time(b) for a, b in fr_pairs)
    full_flops = sum(4 * wl.head_dim * wl.n_q_heads * N * N for N in wl.seq_lens)

    # ---- for comparison: one replica, L2 flushed (256 MiB write) before every call, each call
    # bracketed by its own events (the launch latency after the flush kernel is inside) ----
    flush = torch.empty(256 << 20, dtype=torch.int8, device=dev)
    ctx.build(0, *sched.full[0])
    fl_pairs = []
    for i in range(8 + min(K, 64)):
        _, s, (qb, kb, vb) = sched.step_inputs(i % S)
        flush.add_(1)
        e = (mk(), mk())
        e[0].record(); ctx.step(qb, kb, vb, *outs[0]); e[1].record()
        if i >= 8:
            fl_pairs.append(e)
    torch.cuda.synchronize()
    flush_step_ms = statistics.mean(a.elapsed_time(b) for a, b in fl_pairs)
    del flush
    # ---- for context: a plain device-to-device copy that moves the step kernel's algorithmic bytes (half of
    # them read, half written), under both timing protocols of the step; what a launch of this size can reach ----
    copy_ref = None
    try:
        nb = int(counts["step_attn_bytes"]) // 2
        rc = max(2, min(R, (4 << 30) // max(2 * nb, 1)))
        srcs = [torch.empty(nb, dtype=torch.uint8, device=dev) for _ in range(rc)]
        dsts = [torch.empty(nb, dtype=torch.uint8, device=dev) for _ in range(rc)]
        n_cp = max(4 * rc, 32)
        for i in range(rc):
            dsts[i].copy_(srcs[i])
        torch.cuda.synchronize()
        e0, e1 = mk(), mk()
        e0.record()
        for i in range(n_cp):
            dsts[i % rc].copy_(srcs[i % rc])
        e1.record()
        torch.cuda.synchronize()
        cp_b2b = e0.elapsed_time(e1) / n_cp
        cp_pairs = []
        for i in range(n_cp):
            e = (mk(), mk())
            e[0].record(); dsts[i % rc].copy_(srcs[i % rc]); e[1].record()
            cp_pairs.append(e)
            if i % 4 == 3:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        cp_ev = statistics.mean(a.elapsed_time(b) for a, b in cp_pairs)
        copy_ref = {"bytes": 2 * nb, "back_to_back_us": round(cp_b2b * 1e3, 2), "event_bracketed_us": round(cp_ev * 1e3, 2),
                    "back_to_back_gbs": round(2 * nb / (cp_b2b * 1e-3) / 1e9, 1),
                    "event_bracketed_gbs": round(2 * nb / (cp_ev * 1e-3) / 1e9, 1), "buffers": rc,
                    "how": "torch copy_ between two device buffers of half the step kernel's algorithmic bytes each, "
                           "buffer pairs visited round-robin: context for the fraction above (the measured peak is a "
                           "2 GB copy; a launch of this size cannot reach it), not a denominator"}
        del srcs, dsts
    except Exception as ex:
        sys.stderr.write("same-size copy skipped: %r\n" % (ex,))
    clocks.mark()      # window: the headline repeats, the per-kernel passes, the full recompute and the flushed pass
    clock_info = clocks.stop()

    # ---- warm L2: the same replica stepped K times from one CUDA-graph replay ----
    warm_ms = None
    try:
        gs = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(gs):
            with torch.cuda.graph(graph, stream=gs):
                for i in range(K):
                    _, s, (qb, kb, vb) = sched.step_inputs(i % S)
                    ctx.step(qb, kb, vb, *outs[0], stream=gs)
            for _ in range(3):
                graph.replay()
            gs.synchronize()
            e0, e1 = mk(), mk()
            e0.record(gs); graph.replay(); e1.record(gs)
            gs.synchronize()
            warm_ms = e0.elapsed_time(e1)
    except Exception as ex:   # graph capture is an extra, never the headline
        warm_ms = None
        sys.stderr.write("warm-L2 graph replay skipped: %r\n" % (ex,))
    torch.cuda.synchronize()

    # ---- e2e: host buffers through the *_host entry points, copies inside the timed region ----
    n_e2e = max(8, min(K, 2 * S))
    pin = lambda t: t.cpu().pin_memory()
    h_full = {}
    h_steps = []
    for i in range(n_e2e):
        blk, s, tens = sched.step_inputs(i)
        if s == 0 and blk not in h_full:
            h_full[blk] = tuple(pin(t) for t in sched.full[blk])
        h_steps.append(tuple(pin(t) for t in tens))
    # (two result buffers on the host, alternating: the copy of a step's result runs beside the next step)
    outs_h = [torch.empty(T, wl.n_q_heads, wl.head_dim, dtype=out_t).pin_memory() for _ in range(2)]
    lses_h = [torch.empty(T, wl.n_q_heads).pin_memory() for _ in range(2)]
    ctx.build_host(0, *h_full[0])
    ctx.step_host(*h_steps[0], outs_h[0], lses_h[0])     # allocates staging, warms the path
    torch.cuda.synchronize(); barrier()
    e0, e1 = mk(), mk()
    e0.record()
    n_builds_e2e = 0
    for i in range(n_e2e):
        blk, s, _ = sched.step_inputs(i)
        if s == 0:
            ctx.build_host(blk, *h_full[blk]); n_builds_e2e += 1
        ctx.step_host(*h_steps[i], outs_h[i & 1], lses_h[i & 1])
    ctx.join_host()      # the last result copy, inside the timed region
    e1.record()
    torch.cuda.synchronize(); barrier()
    e2e_ms = e0.elapsed_time(e1)
    el = 2 if wl.dtype == "bf16" else 4
    blk_in = wl.batch * wl.block_len * (wl.n_q_heads + 2 * wl.n_kv_heads) * wl.head_dim * el
    full_in = T * (wl.n_q_heads + 2 * wl.n_kv_heads) * wl.head_dim * el
    h2d = blk_in + full_in * n_builds_e2e / max(n_e2e, 1)
    d2h = T * wl.n_q_heads * wl.head_dim * (2 if out_bf16 else 4) + T * wl.n_q_heads * 4

    for c in range(R):
        st, msg = ctxs[c].poll_status()
        if st != 0:
            raise SystemExit("device status: %s" % msg)

    # ---- reduce over ranks (timing only) ----
    total_ms = reduce_max(total_ms, dev)
    e2e_ms = reduce_max(e2e_ms, dev)
    fr_ms = reduce_max(fr_ms, dev)
    if warm_ms is not None:
        warm_ms = reduce_max(warm_ms, dev)
    value = world * K / (total_ms * 1e-3)

    if rank == 0:
        step_k = statistics.mean(kern_step_ms) * 1e-3
        build_k = statistics.mean(kern_build_ms) * 1e-3 if kern_build_ms else None
        total_flops = K * counts["step_flops"] + n_builds * counts["build_flops"]
        ach = counts["step_attn_bytes"] / step_k / 1e9
        roof = {"kernel": "tc_attn_kernel (step: fixed rows x block keys + merge, block rows x all keys)",
                "bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": round(ach / peaks["hbm_gbs"], 4), "peak_source": peaks["source"],
                "traffic": TRAFFIC_PER_LAUNCH.get((wl.cfg, precision)), "avg_launch_us": round(step_k * 1e6, 2),
                "how": "algorithmic bytes / mean duration of the launch between an event pair recorded inside "
                       "the library (the pair keeps the launch from overlapping its neighbours and contains its "
                       "launch latency)",
                "algorithmic_bytes_per_launch": counts["step_attn_bytes"]}
        if copy_ref:
            roof["copy_of_the_same_bytes"] = copy_ref
        if span:
            a2 = counts["step_attn_bytes"] / (span["step_us"] * 1e-6) / 1e9
            roof["overlapped"] = dict(span, achieved=round(a2, 1), frac=round(a2 / peaks["hbm_gbs"], 4),
                                      step_period_us=round(total_ms / K * 1e3, 2))
        fr_value = world * 1e3 / fr_ms
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": round(total_ms / K, 5), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": "cfg%d %s" % (wl.cfg, wl.name), "batch": wl.batch, "prompt_lens": list(wl.prompt_lens),
                       "gen_len": wl.gen_len, "block_len": wl.block_len, "steps_per_block": S,
                       "heads": "%d/%d" % (wl.n_q_heads, wl.n_kv_heads), "head_dim": wl.head_dim,
                       "precision_mode": precision, "out_dtype": "bf16" if out_bf16 else "f32",
                       "l2": "inputs larger than L2: %d replicas of the cache state visited round-robin "
                             "(%.0f MB of algorithmic traffic between two visits of a replica, L2 is 126 MB), "
                             "calls back to back, no flush" % (R, (R - 1) * counts["step_attn_bytes"] / 1e6)},
            "protocol": {"replicas": R, "builds_in_timed_region": n_builds, "repeats": len(times),
                         "ms_per_repeat": {"median": round(total_ms, 4), "min": round(min(times), 4),
                                           "max": round(max(times), 4)},
                         "launch": launch_mode,
                         "how": "each repeat: untimed pass that puts every replica at its place in its block "
                                "schedule (a build and a step each), barrier + synchronize, K calls (a step each, "
                                "preceded by the block's build where a replica enters a block: round(K / "
                                "steps_per_block) builds) between one event pair, synchronize; value = K / median. "
                                "The K calls are captured once into a CUDA graph (the library's own launches in "
                                "call order, programmatic dependencies included) and each repeat replays it; "
                                "`eager` is the same region with the calls issued one by one from Python",
                         "step_overlap": "on (inputs resident before the first call)",
                         "engine": "tcgen05" if tc else "simt"},
            "eager": None if eager_ms is None else {
                "value": round(world * K / (eager_ms * 1e-3), 1), "unit": UNIT, "step_period_us": round(eager_ms / K * 1e3, 2),
                "how": "the same K calls issued one by one through the Python binding (two kernel launches per step "
                       "from the host; bound by the host's enqueue time when that exceeds the step's device time)"},
            "tflops": round(total_flops / (total_ms * 1e-3) / 1e12, 2),
            "full_recompute": {"value": round(fr_value, 1), "unit": UNIT, "step_us": round(fr_ms * 1e3, 2),
                               "kernel_us": round(fr_kernel_ms * 1e3, 2),
                               "tflops": round(full_flops / (fr_kernel_ms * 1e-3) / 1e12, 1),
                               "tensor_frac": round(full_flops / (fr_kernel_ms * 1e-3) / 1e12 / peaks["bf16_tflops"], 4),
                               "calls": n_fr,
                               "how": "lacache_full_recompute (every row x every key, no cache: the full pass the "
                                      "method replaces) on the same replicas round-robin, calls back to back"},
            "speedup_vs_full_recompute": round(value / fr_value, 3),
            "flushed_l2": {"value": round(world * 1e3 / flush_step_ms, 1), "unit": UNIT,
                           "step_us": round(flush_step_ms * 1e3, 2),
                           "how": "one replica, 256 MiB write before every call, each call bracketed by its own events"},
            "warm_l2": None if warm_ms is None else {
                "value": round(world * K / (warm_ms * 1e-3), 1), "unit": UNIT,
                "how": "one replica stepped K times from one CUDA-graph replay"},
            "roofline": roof,
            "roofline_build": None if build_k is None else {
                "kernel": "tc_attn_kernel (build: fixed rows x fixed keys -> cached state)", "bound": "tensor",
                "achieved": round(counts["build_flops"] / build_k / 1e12, 1), "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s", "frac": round(counts["build_flops"] / build_k / 1e12 / peaks["bf16_tflops"], 4),
                "avg_launch_us": round(build_k * 1e6, 2), "peak_source": peaks["source"]},
            "step_tensor_frac": round(counts["step_flops"] / step_k / 1e12 / peaks["bf16_tflops"], 4),
            # consecutive steps overlap on the device (and launch latency is hidden), so the period of a
            # step in the timed region is shorter than the event-bracketed duration of its attention
            # kernel above; the same algorithmic bytes over that period (builds included in the period):
            "effective": {"step_period_us": round(total_ms / K * 1e3, 2),
                          "hbm_gbs": round(counts["step_bytes"] / (total_ms / K * 1e-3) / 1e9, 1),
                          "hbm_frac": round(counts["step_bytes"] / (total_ms / K * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)},
            "e2e": {"value": round(world * n_e2e / (e2e_ms * 1e-3), 1), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(d2h), "steps": n_e2e},
            "gpu_launches": launches,
            "clocks": clock_info,
            "wall_s_timed_region": round(t_wall, 3),
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(wl, budget_s=12.0)
    for c in ctxs:
        c.destroy()
    if rank == 0 and world == 1 and tc and precision != binding.PRECISION_SPLIT and not args.no_split_leg:
        # the same protocol with the split bf16 planes (the mode that holds for any input): its own contexts
        sctxs = make_replicas(precision_mode=binding.PRECISION_SPLIT)
        srr = RoundRobin(sctxs, outs, sched, min(K, 256), S)
        stimes, _, sbuilds, _ = timed_region(srr, max(3, min(W, 8)), min_ms=20.0)
        sms = statistics.median(stimes)
        spairs = []
        for c in sctxs:
            c.build(0, *sched.full[0])
        for i in range(16):       # event-bracketed step kernel, as for the headline's roofline
            e = (mk(), mk()); e[0].record(); e[1].record()
            c = sctxs[i % R]
            c.set_timing_events(*e); spairs.append(e)
            _, s_, (qb, kb, vb) = sched.step_inputs(i % S)
            c.step(qb, kb, vb, *outs[i % R])
        torch.cuda.synchronize()
        skern = statistics.mean(a.elapsed_time(b) for a, b in spairs) * 1e-3
        for c in sctxs:
            c.set_timing_events(None, None)
            st, msg = c.poll_status()
            if st != 0:
                raise SystemExit("device status (split-operands leg): %s" % msg)
            c.destroy()
        line["split_operands"] = {"value": round(srr.K / (sms * 1e-3), 1), "unit": UNIT, "steps": srr.K,
                                  "step_period_us": round(sms / srr.K * 1e3, 2), "builds_in_timed_region": sbuilds,
                                  "repeats": len(stimes), "step_kernel_us": round(skern * 1e6, 2),
                                  "roofline_frac": round(counts["step_attn_bytes"] / skern / 1e9 / peaks["hbm_gbs"], 4),
                                  "how": "precision_mode = split (two bf16 planes per operand, three score products; "
                                         "holds the tolerance for any input): same round-robin protocol"}
    if rank == 0 and world == 1 and tc and not args.no_tile_granular and wl.total_tokens <= 65536:
        # Algorithm 1 at tile granularity (less cached, more step work): the same protocol, its own contexts
        tctxs = make_replicas(cache_granularity=binding.GRANULARITY_TILE)
        trr = RoundRobin(tctxs, outs, sched, min(K, 256), S)
        ttimes, _, tbuilds, _ = timed_region(trr, max(3, min(W, 8)), min_ms=20.0)
        tms = statistics.median(ttimes)
        for c in tctxs:
            st, msg = c.poll_status()
            if st != 0:
                raise SystemExit("device status (tile-granular leg): %s" % msg)
            c.destroy()
        line["tile_granular"] = {"value": round(trr.K / (tms * 1e-3), 1), "unit": UNIT, "steps": trr.K,
                                 "step_period_us": round(tms / trr.K * 1e3, 2), "builds_in_timed_region": tbuilds,
                                 "repeats": len(ttimes), "vs_token_granular": round(trr.K / (tms * 1e-3) / value, 3),
                                 "how": "cache_granularity = tile (state cached only for 128-row tiles and over 128-key "
                                        "tiles that do not overlap the block; Algorithm 1's overlap predicates): same "
                                        "round-robin protocol, same out / lse"}
    del outs, sched
    if rank == 0:
        if (world == 1 and not args.no_token_path and wl.dtype == "bf16" and wl.n_q_heads in D_MODEL
                and wl.total_tokens <= 65536 and not out_bf16):
            line["token_path"] = token_path_leg(wl, dev, peaks, args.seed, min(K, 512), precision)
        if world == 1 and not args.no_sampler and wl.n_q_heads in VOCAB and wl.total_tokens * VOCAB[wl.n_q_heads] * 2 <= 8e9:
            line["sampler"] = sampler_leg(wl, dev, peaks, args.seed)
        if (world == 1 and not args.no_incremental and wl.dtype == "bf16" and wl.head_dim == 128 and wl.n_blocks >= 2
                and not out_bf16):
            line["incremental"] = incremental_leg(wl, dev, args.seed, R, precision)
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ----------------------------------------------------------------------------
# sampling-stage truncation: softmax over the vocabulary on the current block's rows only
# ----------------------------------------------------------------------------
VOCAB = {32: 126464, 28: 152064}     # vocabulary of the model a workload is shaped like, by query heads
SAMPLER_TRAFFIC_PER_LAUNCH = {4: 66288640}   # ncu, profiles/sample_rows_kernel_cfg4_ncu_full.txt (read + write)


def sampler_leg(wl, dev, peaks, seed):
    """Device time of lacache_sample_block on bf16 logits [T, vocab] (synthetic, N(0, 3)).  Headline: calls
    back to back over replicas of the logits array whose block rows together exceed L2 twice over, one event
    pair around all of them.  Also: one call after a 256 MiB write, bracketed by its own events (every
    access of its dependent chain cold); the median.  Algorithmic bytes = block rows x vocab x 2."""
    import torch
    from paper_2607_16339_b200 import binding
    from paper_2607_16339_b200.workloads import DeviceSchedule
    mk = lambda: torch.cuda.Event(enable_timing=True)
    V, T, n = VOCAB[wl.n_q_heads], wl.total_tokens, wl.batch * wl.block_len
    g = torch.Generator(device=dev).manual_seed(seed + 5)
    sched = DeviceSchedule(wl, seed + 6, dev, 1)
    ctx = binding.Context.from_workload(wl)
    ctx.build(0, *sched.full[0])
    cu = wl.cu_seqlens
    rows = torch.cat([torch.arange(cu[b] + P, cu[b] + P + wl.block_len) for b, P in enumerate(wl.prompt_lens)]).to(dev)
    nbytes = n * V * 2
    # replicas of the logits array visited round-robin: together their block rows exceed L2 twice over
    # (only the block's rows are ever read, so only those are filled)
    R = max(2, -(-2 * L2_BYTES // nbytes) + 1)
    while R > 2 and R * T * V * 2 > 40e9:
        R -= 1
    reps = []
    for _ in range(R):
        lg = torch.empty(T, V, device=dev, dtype=torch.bfloat16)
        for lo in range(0, n, 256):
            lg[rows[lo:lo + 256]] = (torch.randn(min(256, n - lo), V, generator=g, device=dev) * 3).to(torch.bfloat16)
        reps.append(lg)
    conf = torch.empty(n, device=dev); tok = torch.empty(n, device=dev, dtype=torch.int32); lse = torch.empty(n, device=dev)
    for i in range(R):
        ctx.sample_block(reps[i], conf, tok, lse)
    ncalls = max(3 * R, 48)
    e0, e1 = mk(), mk()
    torch.cuda.synchronize()
    e0.record()
    for i in range(ncalls):
        ctx.sample_block(reps[i % R], conf, tok, lse)
    e1.record()
    torch.cuda.synchronize()
    period_us = e0.elapsed_time(e1) * 1e3 / ncalls
    logits = reps[0]
    flush = torch.empty(256 << 20, device=dev, dtype=torch.int8)
    times = []
    for i in range(3 + 21):
        flush.add_(1)
        e = (mk(), mk())
        e[0].record()
        ctx.sample_block(logits, conf, tok, lse)
        e[1].record()
        torch.cuda.synchronize()
        if i >= 3:
            times.append(e[0].elapsed_time(e[1]) * 1e3)
    st, msg = ctx.poll_status()
    if st != 0:
        raise SystemExit("bench.py: device status %d in the sampler leg: %s" % (st, msg))
    ctx.destroy()
    cold_us = sorted(times)[len(times) // 2]
    gbs = nbytes / (period_us * 1e-6) / 1e9
    return {"what": "lacache_sample_block: softmax over the vocabulary on the current block's rows only (token, "
                    "probability, log normaliser), bf16 logits; %d logits arrays visited round-robin, calls back "
                    "to back (launch_us); and one call after a 256 MiB write, bracketed by its own events "
                    "(cold_launch_us)" % R,
            "rows": n, "of_rows": T, "vocab": V, "launch_us": round(period_us, 2), "cold_launch_us": round(cold_us, 2),
            "replicas": R,
            "roofline": {"kernel": "sample_rows_kernel", "bound": "hbm", "achieved": round(gbs, 1),
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(gbs / peaks["hbm_gbs"], 4),
                         "peak_source": peaks["source"], "traffic": SAMPLER_TRAFFIC_PER_LAUNCH.get(wl.cfg),
                         "avg_launch_us": round(period_us, 2), "algorithmic_bytes_per_launch": nbytes}}


# ----------------------------------------------------------------------------
# one whole generation, the cache rebuilt for every block or advanced from block to block
# ----------------------------------------------------------------------------
def incremental_leg(wl, dev, seed, R, precision):
    """Steps per second over one generation (every block, every step of it) of R independent cache
    states visited round-robin, twice: with lacache_build at the start of every block, and with
    lacache_build_incremental at block 0 and lacache_build_advance between blocks.  Also the mean
    device time of one rebuild and of one advance (events around the calls)."""
    import torch
    from paper_2607_16339_b200 import binding
    from paper_2607_16339_b200.workloads import DeviceSchedule
    mk = lambda: torch.cuda.Event(enable_timing=True)
    S, nb, T = wl.steps_per_block, wl.n_blocks, wl.total_tokens
    sched = DeviceSchedule(wl, seed + 17, dev, nb * S)
    ctxs = [binding.Context.from_workload(wl, precision_mode=precision) for _ in range(R)]
    for c in ctxs:
        c.set_step_overlap(True)     # the step inputs are all resident before the first call
    outs = [(torch.empty(T, wl.n_q_heads, wl.head_dim, device=dev), torch.empty(T, wl.n_q_heads, device=dev))
            for _ in range(R)]
    res = {}
    for mode in ("rebuild", "advance", "rebuild", "advance"):     # (the first pass of each warms up)
        pairs = []
        e0, e1 = mk(), mk()
        torch.cuda.synchronize()
        e0.record()
        for b in range(nb):
            for c in range(R):
                ev = (mk(), mk())
                ev[0].record()
                if mode == "rebuild":
                    ctxs[c].build(b, *sched.full[b])
                elif b == 0:
                    ctxs[c].build_incremental(0, *sched.full[0])
                else:
                    ctxs[c].build_advance(*sched.steps[b * S - 1])
                ev[1].record()
                if b > 0:
                    pairs.append(ev)
            for s in range(S):
                for c in range(R):
                    ctxs[c].step(*sched.steps[b * S + s], *outs[c])
        e1.record()
        torch.cuda.synchronize()
        for c in ctxs:
            st, msg = c.poll_status()
            if st != 0:
                raise SystemExit("bench.py: device status %d in the incremental leg: %s" % (st, msg))
        ms = e0.elapsed_time(e1)
        res[mode] = (R * nb * S / (ms * 1e-3), sum(a.elapsed_time(b_) for a, b_ in pairs) / len(pairs) * 1e3)
    for c in ctxs:
        c.destroy()
    return {"what": "one generation of %d blocks x %d steps on %d cache states round-robin: lacache_build per block "
                    "against lacache_build_incremental + lacache_build_advance" % (nb, S, R),
            "value": round(res["advance"][0], 1), "rebuild_value": round(res["rebuild"][0], 1), "unit": UNIT,
            "advance_us": round(res["advance"][1], 1), "rebuild_us": round(res["rebuild"][1], 1),
            "blocks": nb, "steps": R * nb * S, "replicas": R}


# ----------------------------------------------------------------------------
# the step fed by token ids: embedding gather + RMS norm + Q/K/V projection in front
# ----------------------------------------------------------------------------
D_MODEL = {32: 4096, 28: 3584}     # first-layer width of the model a workload is shaped like, by query heads
QKV_TRAFFIC_PER_LAUNCH = {2: 104751872}   # ncu, profiles/qkv_gemm_kernel_cfg2_step_ncu_full.txt


def token_path_leg(wl, dev, peaks, seed, n_steps, precision):
    """Steps per second of lacache_step_tokens (token ids in, attention output out) and the
    event-timed duration of its projection kernel, which is bound by reading the stacked
    Q/K/V weight once per step.  Weight and cache-state replicas are visited round-robin so
    that every call finds them in HBM."""
    import numpy as np
    import torch
    from paper_2607_16339_b200 import binding
    from paper_2607_16339_b200.workloads import TokenModel
    mk = lambda: torch.cuda.Event(enable_timing=True)
    tm = TokenModel(wl, D_MODEL[wl.n_q_heads], 8192, seed)
    T, nb, S = wl.total_tokens, wl.batch * wl.block_len, wl.steps_per_block
    bf = lambda a: torch.from_numpy(a).to(dev).to(torch.bfloat16).contiguous()
    emb, nw, w0 = bf(tm.embed), bf(tm.norm_weight), bf(tm.w_qkv)
    w_bytes = w0.numel() * 2
    R = max(3, -(-2 * L2_BYTES // w_bytes) + 1)
    prods = [binding.QkvProducer(emb, nw, w0, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, tm.rms_eps, T)
             for _ in range(R)]      # each handle holds its own re-laid-out copy of the weight
    ctxs = [binding.Context.from_workload(wl, precision_mode=precision) for _ in range(R)]
    for c in ctxs:
        c.set_step_overlap(True)     # the token ids are all resident before the first call
    out = torch.empty(T, wl.n_q_heads, wl.head_dim, device=dev)
    lse = torch.empty(T, wl.n_q_heads, device=dev)
    blk = wl.n_blocks // 2
    ids_full = torch.from_numpy(tm.full_ids(blk)).to(dev)
    ids_blk = [torch.from_numpy(tm.block_ids(blk, s)).to(dev) for s in range(1, S + 1)]
    for c in range(R):
        ctxs[c].build_tokens(prods[c], blk, token_ids=ids_full)
    torch.cuda.synchronize()
    e0, e1 = mk(), mk()
    e0.record()
    for i in range(2 * R):
        ctxs[i % R].build_tokens(prods[i % R], blk, token_ids=ids_full)
    e1.record(); torch.cuda.synchronize()
    build_us = e0.elapsed_time(e1) / (2 * R) * 1e3
    # the build of the next block that re-projects only the block just finished
    rows_prev = torch.from_numpy(np.concatenate(
        [wl.cu_seqlens[s] + P + (blk - 1) * wl.block_len + np.arange(wl.block_len)
         for s, P in enumerate(wl.prompt_lens)]).astype("int32")).to(dev)
    ids_prev = ids_full[rows_prev.long()].contiguous()
    for c in range(R):
        ctxs[c].build_tokens_update(prods[c], blk, rows_prev, token_ids=ids_prev)
    torch.cuda.synchronize()
    e0.record()
    for i in range(2 * R):
        ctxs[i % R].build_tokens_update(prods[i % R], blk, rows_prev, token_ids=ids_prev)
    e1.record(); torch.cuda.synchronize()
    update_us = e0.elapsed_time(e1) / (2 * R) * 1e3
    launches = 0
    for i in range(16):
        ctxs[i % R].step_tokens(prods[i % R], out, lse, blk_token_ids=ids_blk[i % S])
    torch.cuda.synchronize()
    e0.record()
    for i in range(n_steps):
        ctxs[i % R].step_tokens(prods[i % R], out, lse, blk_token_ids=ids_blk[i % S])
        launches += ctxs[i % R].last_launch_count
    e1.record(); torch.cuda.synchronize()
    step_us = e0.elapsed_time(e1) / n_steps * 1e3
    # the projection kernel alone, event pair recorded inside the library around its launch
    pairs = []
    for i in range(min(n_steps, 96)):
        e = (mk(), mk()); e[0].record(); e[1].record()
        prods[i % R].set_timing_events(*e); pairs.append(e)
        ctxs[i % R].step_tokens(prods[i % R], out, lse, blk_token_ids=ids_blk[i % S])
    torch.cuda.synchronize()
    gemm_us = statistics.mean(a.elapsed_time(b) for a, b in pairs) * 1e3
    for o in prods + ctxs:
        st, msg = o.poll_status()
        if st != 0:
            raise SystemExit("device status (token path): %s" % msg)
        o.destroy()
    d_model = tm.d_model
    alg = w_bytes + nb * d_model * 2 + nb * (wl.n_q_heads + 2 * wl.n_kv_heads) * wl.head_dim * 2
    ach = alg / (gemm_us * 1e-6) / 1e9
    return {
        "what": "lacache_step_tokens: token ids -> embedding gather + RMS norm + Q/K/V projection (tcgen05, stream-K) "
                "-> RoPE + cached attention; synthetic first-layer weights",
        "d_model": d_model, "tokens_per_step": nb, "replicas": R,
        "value": round(1e6 / step_us, 1), "unit": UNIT, "step_us": round(step_us, 2),
        "build_tokens_us": round(build_us, 1), "build_tokens_update_us": round(update_us, 1),
        "gpu_launches": launches, "steps": n_steps,
        "roofline": {"kernel": "qkv_gemm_kernel (one step: %d tokens x %d -> %d features)" % (nb, d_model, w0.shape[0]),
                     "bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": round(ach / peaks["hbm_gbs"], 4), "peak_source": peaks["source"],
                     "traffic": QKV_TRAFFIC_PER_LAUNCH.get(wl.cfg), "avg_launch_us": round(gemm_us, 2),
                     "algorithmic_bytes_per_launch": int(alg)},
    }


# per-launch DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the
# step attention kernel from the committed ncu captures
# (profiles/tc_attn_kernel_cfg2_ncu_full.txt, tc_attn_kernel_cfg{3,4}_step_ncu_full.txt,
# tc_attn_kernel_cfg5_{split,plain}_ncu_full.txt), bytes; None where no capture exists for the workload
# and precision mode.  The fp32 output (12.6 MB) is still in L2 when the
# kernel ends, so the figure is dominated by reads.
DEFAULT_PRECISION = {1: 1, 2: 3, 3: 1, 4: 3, 5: 3, 6: 3}   # binding.PRECISION_*: 1 = split bf16 planes, 3 = one fp16 plane
TRAFFIC_PER_LAUNCH = {(2, 1): 48370432, (3, 1): 93736960, (4, 1): 460605952, (5, 1): 209015552, (5, 0): 161659392,
                      (2, 3): 34980608, (4, 3): 345821952, (5, 3): 161281536}   # (config, precision mode)


# ----------------------------------------------------------------------------
# the CPU oracle, timed (baseline / reference arm)
# ----------------------------------------------------------------------------
def cpu_baseline(wl, budget_s=12.0, max_steps=64):
    import numpy as np
    import oracle
    from paper_2607_16339_b200.workloads import SyntheticSchedule
    sch = SyntheticSchedule(wl, seed=0)
    sch.begin_block(0)
    scale = wl.head_dim ** -0.5
    n, t_total = 0, 0.0
    rows = None
    # one untimed pass sizes the sample
    t0 = time.perf_counter()
    stride = 1
    if wl.total_tokens * wl.total_tokens * wl.n_q_heads > 4e8:
        stride = 8
    rows = np.arange(0, wl.total_tokens, stride, dtype=np.int32)
    sch.draw_step(0, 1)
    oracle.attention(sch.q, sch.k, sch.v, wl.cu_seqlens, wl.rope_theta, scale, rows=rows)
    t_one = time.perf_counter() - t0
    reps = int(max(1, min(max_steps, budget_s / max(t_one, 1e-3))))
    for s in range(reps):
        sch.draw_step(0, 1 + s % wl.steps_per_block)
        t0 = time.perf_counter()
        oracle.attention(sch.q, sch.k, sch.v, wl.cu_seqlens, wl.rope_theta, scale, rows=rows)
        t_total += time.perf_counter() - t0
        n += 1
    frac = len(rows) / wl.total_tokens
    return {"value": round(n * frac / t_total, 4), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "%d evaluations of the fp64 full-sequence definition on cfg%d, %d of %d query rows each "
                      "(all heads, all keys); value scaled by the row fraction" % (n, wl.cfg, len(rows), wl.total_tokens)}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2607_16339_b200.workloads import WORKLOADS, SyntheticSchedule
    wl = WORKLOADS[args.workload]
    K, W = args.steps, args.warmup
    sch = SyntheticSchedule(wl, seed=0)
    sch.begin_block(0)
    scale = wl.head_dim ** -0.5
    # bounded sample: a strided subset of the query rows per step so that K + W
    # steps finish within a few minutes; the value is scaled by the row fraction
    budget = 150.0
    t0 = time.perf_counter()
    sch.draw_step(0, 1)
    probe_rows = np.arange(0, wl.total_tokens, 16, dtype=np.int32)
    oracle.attention(sch.q, sch.k, sch.v, wl.cu_seqlens, wl.rope_theta, scale, rows=probe_rows)
    t_probe = time.perf_counter() - t0
    per_row = t_probe / len(probe_rows)
    rows_per_step = int(max(8, min(wl.total_tokens, budget / ((K + W) * per_row))))
    stride = max(1, wl.total_tokens // rows_per_step)
    rows = np.arange(0, wl.total_tokens, stride, dtype=np.int32)
    times = []
    for i in range(W + K):
        sch.draw_step((i // wl.steps_per_block) % wl.n_blocks, 1 + i % wl.steps_per_block)
        t0 = time.perf_counter()
        oracle.attention(sch.q, sch.k, sch.v, wl.cu_seqlens, wl.rope_theta, scale, rows=rows)
        if i >= W:
            times.append(time.perf_counter() - t0)
    frac = len(rows) / wl.total_tokens
    total = sum(times)
    value = K * frac / total
    sample = ("fp64 full-sequence definition, %d of %d query rows per step (stride %d), all heads and keys; "
              "value scaled by the row fraction" % (len(rows), wl.total_tokens, stride))
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": round(total / K / frac * 1e3, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "cfg%d %s" % (wl.cfg, wl.name), "batch": wl.batch, "prompt_lens": list(wl.prompt_lens),
                       "gen_len": wl.gen_len, "block_len": wl.block_len, "steps_per_block": wl.steps_per_block,
                       "heads": "%d/%d" % (wl.n_q_heads, wl.n_kv_heads), "head_dim": wl.head_dim},
            "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--workload", type=int, default=2, help="config number 1..6 (2 = the headline LLaDA-8B shape; 6 = the large-batch extension)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-token-path", action="store_true", help="skip the extra leg that feeds steps from token ids")
    ap.add_argument("--no-sampler", action="store_true", help="skip the extra leg that times the sampling-stage truncation")
    ap.add_argument("--no-incremental", action="store_true",
                    help="skip the extra leg that compares rebuilding the cache per block with advancing it")
    ap.add_argument("--replicas", type=int, default=0, help="cache-state replicas visited round-robin (0 = sized from the L2)")
    ap.add_argument("--no-split-leg", action="store_true", help="skip the extra leg with split bf16 operands")
    ap.add_argument("--no-tile-granular", action="store_true", help="skip the extra leg with tile-granular caching")
    ap.add_argument("--precision-mode", type=int, default=-1,
                    help="0 = one bf16 plane per operand (suits the small-score configurations 5 and 6), 1 = split bf16 planes (any input), 3 = one fp16 plane (default except for configuration 3, whose outlier keys need the split)")
    ap.add_argument("--out-dtype", default="f32", choices=["f32", "bf16"])
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
