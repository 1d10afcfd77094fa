"""Benchmark of the per-layer KV-cache eviction pass (prefix tokens evicted per second per layer).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg4|cfg3|cfg2] [--budget B]
    python bench.py --impl reference ...      # the fp64 CPU oracle, timed on the host cores

One step = one pass of the whole hot path (scores -> pool -> top-k -> gather) over every layer of
one synthetic cache, on one stream.  Every (layer, KV head) is an independent unit of the pass, so the
layers of a cache are evicted by ONE call: jq_evict_layers on the layers' own buffers (`--call layers`,
the default), or jq_evict_layer on tensors that stack the layers along the KV-head axis (`--call stacked`);
the same work as one call per layer (`--call per-layer`) is also timed and reported.  The ragged batch
(`--workload cfg4`: four sequences of different lengths, 32 layers each) is one jq_evict_ragged call per step.
Every step is bracketed by CUDA events on the launching stream; `value` comes from the time of all K steps
(first to last event), the median step is reported beside it.  Prints ONE JSON line.
With N > 1 (torchrun) every rank evicts a cache of its own (independent replicas, no collective on
the data path); the value is the sum over ranks divided by the slowest rank's time.
"""
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

import jq_workloads as W  # noqa: E402

METRIC = "prefix tokens evicted/sec per layer"
# dram__bytes_read.sum + dram__bytes_write.sum of one score_fused launch on one layer (ncu, see profiles/);
# to be emptied when the kernel changes after the counters were taken
NCU_DRAM_BYTES_PER_LAYER = {"cfg5-llama8b-128k": 357.0e6, "cfg3-llama8b-32k-32layers": 68.5e6}
UNIT = "tokens/s"
SM_MAX_MHZ = 1965.0


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--fma-compare", action="store_true", help="also time the CUDA-core comparator of the scoring step")
    ap.add_argument("--decode", action="store_true", help="also time one decoding step over a layer's pruned cache")
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=["cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--seq", type=int, default=None,
                    help="cfg4 only: time one sequence of the ragged batch (0..3) instead of the whole batch in one call")
    ap.add_argument("--budget", type=int, default=None)
    ap.add_argument("--layers", type=int, default=None, help="layer calls per step (default: the workload's)")
    ap.add_argument("--call", default="layers", choices=["layers", "stacked", "per-layer"],
                    help="layers: one jq_evict_layers call per step on per-layer buffers (default); stacked: one jq_evict_layer call on "
                         "layers concatenated along the KV-head axis; per-layer: one jq_evict_layer call per layer")
    ap.add_argument("--windowed", action="store_true",
                    help="window-inclusive scoring (jq_evict_layer_windowed): the causal keys of the query positions join the softmax")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the second target cache (the 32K-key workload) of the default line")
    return ap.parse_args()


def pick_workload(args):
    wl = {"cfg2": W.CFG2, "cfg3": W.CFG3, "cfg4": W.CFG4[(args.seq if args.seq is not None else 3) % 4], "cfg5": W.CFG5}[args.workload]
    if args.workload == "cfg2":
        wl = W.Workload(wl.name, 2, wl.Hkv, wl.Hq, wl.L, wl.w, wl.budget, layers=32, distinct_layers=32)
    if args.budget:
        wl = wl.with_budget(args.budget)
    return wl


CALLS = {"stacked": "one jq_evict_layer call per step, the layers stacked along the KV-head axis",
         "layers": "one jq_evict_layers call per step, every layer in buffers of its own",
         "ragged": "one jq_evict_ragged call per step: every (sequence, layer) a unit with buffers, length and budget of its own",
         "per-layer": "one jq_evict_layer call per layer",
         "oracle": "the CPU oracle on a bounded sample of one layer"}


def config_of(wl, layers, distinct, call="per-layer"):
    return {"workload": wl.name, "L": wl.L, "Hkv": wl.Hkv, "Hq": wl.Hq, "d": wl.d, "w": wl.w,
            "budget": wl.budget, "pool": wl.pool, "layers_per_step": layers, "distinct_layers": distinct,
            "call": CALLS[call],
            "l2": "inputs larger than L2 (K of one step: %.0f MiB)" % (layers * wl.Hkv * wl.L * wl.d * 2 / 2**20)}


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_time_heads(wl, K, V, Q, heads):
    """Seconds the oracle takes for the whole pass restricted to the given KV heads (independent units)."""
    import oracle
    g = wl.group
    qrows = np.concatenate([np.arange(kv * g, kv * g + g) for kv in heads])
    Ks, Vs, Qs = np.ascontiguousarray(K[heads]), np.ascontiguousarray(V[heads]), np.ascontiguousarray(Q[qrows])
    t0 = time.perf_counter()
    oracle.evict_layer(Ks, Vs, Qs, wl.budget, wl.pool)
    return time.perf_counter() - t0


def cpu_baseline(wl, K, V, Q, max_heads=None):
    import oracle
    cores = os.cpu_count() or 1
    n = min(wl.Hkv, cores if max_heads is None else max_heads)
    heads = list(range(n))
    sec = oracle_time_heads(wl, K, V, Q, heads)
    t_layer = sec * wl.Hkv / n
    return {"value": wl.L / t_layer, "unit": UNIT, "cores": oracle.threads(n), "kind": "oracle",
            "sample": "%d of %d KV heads of one layer at full L=%d (heads are independent); %.2f s measured, "
                      "scaled to a layer; gcc -O2 -fopenmp, fp64" % (n, wl.Hkv, wl.L, sec),
            "seconds_per_layer": t_layer}


def run_reference(args):
    """The reference arm: the fp64 oracle as it stands, on the host cores, rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    wl = pick_workload(args)
    K, V, Q, _ = W.make_layer(wl, 0)
    cores = os.cpu_count() or 1
    # calibrate on a short prefix with the heads a step runs (in parallel, as in a step), then size the per-step
    # sample so that the whole run takes about two minutes
    n = max(1, min(wl.Hkv, cores))
    heads = list(range(n))
    Lc = max(wl.L // 16, 256)
    wc = wl.with_L(Lc)
    tc = oracle_time_heads(wc, np.ascontiguousarray(K[:, :Lc]), np.ascontiguousarray(V[:, :Lc]), Q, heads)
    per_step = tc * wl.L / Lc
    total = args.steps + args.warmup
    Ls = wl.L
    if total * per_step > 100.0:
        Ls = max(2048, int(wl.L * 100.0 / (total * per_step)) // 128 * 128)
    ws = wl.with_L(Ls)
    Ks, Vs = np.ascontiguousarray(K[:, :Ls]), np.ascontiguousarray(V[:, :Ls])
    for _ in range(args.warmup):
        oracle_time_heads(ws, Ks, Vs, Q, heads)
    t = [oracle_time_heads(ws, Ks, Vs, Q, heads) for _ in range(args.steps)]
    sec = float(np.mean(t))
    t_layer = sec * (wl.Hkv / n) * (wl.L / Ls)
    value = wl.L / t_layer
    sample = "%d of %d KV heads, first %d of %d keys, per step; scaled linearly to a full layer" % (n, wl.Hkv, Ls, wl.L)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, 1, 1, "oracle"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(n), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- N > 1: independent replicas

def max_over_ranks(ms, world, device="cuda"):
    """The job's time is the slowest rank's: all-reduce MAX of the rank-local milliseconds (no-op at N = 1)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(wl, world, t_layer):
    """Whole-job throughput: every rank evicts a cache of its own (replicas, no data-path collective)."""
    return world * wl.L / t_layer


# ----------------------------------------------------------------------------- GPU arm

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.f.read().strip().splitlines():
            c = [x.strip() for x in ln.split(",")]
            if len(c) < 7:
                continue
            try:
                sm.append(float(c[0])); mx.append(float(c[1])); pw.append(float(c[2]))
            except ValueError:
                continue
            for nm, v in zip(names, c[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), power_w_max=float(max(pw)),
                       reasons=sorted(reasons), samples=len(sm))
        return out


class Timer:
    """Steps on one stream with a CUDA event between consecutive steps, the SM clock sampled meanwhile."""

    def __init__(self, torch, stream, barrier, gpu_index, sample_clocks):
        self.torch, self.stream, self.barrier, self.gpu, self.sample = torch, stream, barrier, gpu_index, sample_clocks

    def run(self, step, steps, warmup=3, min_seconds=0.0):
        """Returns (total ms of `steps` steps, list of per-step ms, clocks).  With min_seconds the step count is raised so
        that the region lasts long enough for the clock sampler to see it (the count actually run is len(per-step))."""
        torch = self.torch
        for _ in range(warmup):
            step()
        self.barrier()
        if min_seconds > 0:
            e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            e[0].record(self.stream); step(); e[1].record(self.stream)
            torch.cuda.synchronize()
            steps = max(steps, int(min_seconds * 1e3 / max(e[0].elapsed_time(e[1]), 1e-3)) + 1)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        sampler = ClockSampler(self.gpu) if self.sample else None
        if sampler:
            time.sleep(0.05)
        ev[0].record(self.stream)
        for i in range(steps):
            step()
            ev[i + 1].record(self.stream)
        self.barrier()
        clocks = sampler.stop() if sampler else None
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        return ev[0].elapsed_time(ev[steps]), per, clocks


def kcycles(ms, clocks):
    """Thousands of SM cycles a duration corresponds to at the clock sampled while it ran (None without samples)."""
    if not clocks or not clocks.get("sm_mhz"):
        return None
    return ms * clocks["sm_mhz"]


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2509_10798_b200 as jq

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    jq.lib()                                   # fails loudly if the CUDA library is not built

    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    timer = Timer(torch, stream, barrier, local, rank == 0)

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    def device_layers(wl, layers, distinct, seq):
        """The layers of a cache as a cache holds them: a tensor each (a layer the workload repeats gets a copy of its own)."""
        Ks, Vs, Qs, host0 = [], [], [], None
        for i in range(distinct):
            K, V, Q, _ = W.make_layer(wl, layer=i, seq=seq)
            if i == 0:
                host0 = (K, V, Q)
            Ks.append(dev(K)); Vs.append(dev(V)); Qs.append(dev(Q))
        for i in range(distinct, layers):
            Ks.append(Ks[i % distinct].clone()); Vs.append(Vs[i % distinct].clone()); Qs.append(Qs[i % distinct].clone())
        return Ks, Vs, Qs, host0

    def one_call_cache(wl, layers, distinct, seq, steps, min_seconds=0.0):
        """Times jq_evict_layers on a cache of `layers` layers of workload wl: per-layer time, clocks, stage times."""
        s = jq.shape(wl.Hkv, wl.Hq, wl.L, wl.w, wl.budget, wl.pool, wl.d)
        Ks, Vs, Qs, _ = device_layers(wl, layers, distinct, seq)
        Ko = torch.zeros((wl.Hkv * layers, wl.nkeep, wl.d), dtype=torch.bfloat16, device="cuda")
        Vo = torch.zeros_like(Ko)
        idx = torch.zeros((wl.Hkv * layers, wl.nkeep), dtype=torch.int32, device="cuda")
        ws = jq.new_layers_workspace(s, layers)
        total, per, clocks = timer.run(lambda: jq.evict_layers(Ks, Vs, Qs, s, Ko, Vo, idx, ws, stream=stream), steps, min_seconds=min_seconds)
        assert jq.last_device_status(ws) == jq.JQ_OK, "device status not ok"
        t_layer = max_over_ranks(total, world) * 1e-3 / (len(per) * layers)
        gbs = W.formula_bytes(wl) / t_layer / 1e9
        return {"workload": wl.name, "L": wl.L, "w": wl.w, "budget": wl.budget, "layers_per_step": layers, "distinct_layers": distinct,
                "call": CALLS["layers"], "steps": len(per), "ms_per_layer": t_layer * 1e3,
                "ms_per_layer_median": float(np.median(per)) / layers, "value": job_value(wl, world, t_layer), "unit": UNIT,
                "layer_formula_gbs": gbs, "layer_frac_of_8tbs": gbs / 8000.0, "clocks": clocks,
                "kcycles_per_layer": kcycles(t_layer * 1e3, clocks)}

    wl = pick_workload(args)
    ragged = args.workload == "cfg4" and args.seq is None
    layers = args.layers or wl.layers
    distinct = min(wl.distinct_layers, layers)
    if ragged:
        distinct = min(distinct, 2)            # two generated layers per sequence, the rest device copies (a step moves the same bytes)
    s = jq.shape(wl.Hkv, wl.Hq, wl.L, wl.w, wl.budget, wl.pool, wl.d)
    nkeep = wl.nkeep

    if ragged:
        # the whole ragged batch in ONE call: unit = (sequence, layer)
        seqs = [w.with_budget(args.budget) if args.budget else w for w in W.CFG4]
        RK, RV, RQ, RL, RB = [], [], [], [], []
        host0 = None
        for q, wq in enumerate(seqs):
            Kq, Vq, Qq, h0 = device_layers(wq, layers, distinct, q)
            if q == 3:
                host0 = h0
            RK += Kq; RV += Vq; RQ += Qq; RL += [wq.L] * layers; RB += [wq.budget] * layers
        rows = jq.ragged_output_rows(s, len(RK), RL, RB)
        KoR = torch.zeros((rows, wl.d), dtype=torch.bfloat16, device="cuda")
        VoR = torch.zeros_like(KoR)
        idxR = torch.zeros((rows,), dtype=torch.int32, device="cuda")
        wsR = jq.new_ragged_workspace(s, len(RK), RL)
        tokens_per_layer = sum(w.L for w in seqs)
        bytes_per_layer = sum(W.formula_bytes(w) for w in seqs)

        def step():
            jq.evict_ragged(RK, RV, RQ, s, RL, RB, KoR, VoR, idxR, wsR, stream=stream)
        call = "ragged"
        Ks, Vs, Qs = RK[3 * layers:], RV[3 * layers:], RQ[3 * layers:]      # the longest sequence, for the per-layer comparison
    else:
        Ks, Vs, Qs, host0 = device_layers(wl, layers, distinct, rank)
        Kws = [dev(W.make_window_keys(wl, host0[2] if i == 0 else W.make_layer(wl, layer=i % distinct, seq=rank)[2], layer=i % distinct, seq=rank))
               for i in range(layers)] if args.windowed else []
        tokens_per_layer = wl.L
        bytes_per_layer = W.formula_bytes(wl)
        call = args.call
        if args.windowed and call == "layers":
            call = "stacked"          # the window-inclusive entry point takes one (stacked) tensor per operand
    ws = jq.new_workspace(s)
    Ko = torch.zeros((wl.Hkv, nkeep, wl.d), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.zeros((wl.Hkv, nkeep), dtype=torch.int32, device="cuda")

    def step_per_layer():
        for i in range(layers):
            if args.windowed:
                jq.evict_layer_windowed(Ks[i], Vs[i], Qs[i], Kws[i], s, Ko, Vo, idx, ws, stream=stream)
            else:
                jq.evict_layer(Ks[i], Vs[i], Qs[i], s, Ko, Vo, idx, ws, stream=stream)

    sS = jq.shape(wl.Hkv * layers, wl.Hq * layers, wl.L, wl.w, wl.budget, wl.pool, wl.d)
    one_call = ragged or call in ("stacked", "layers")
    if not ragged:
        KoS = torch.zeros((sS.Hkv, nkeep, wl.d), dtype=torch.bfloat16, device="cuda")
        VoS = torch.zeros_like(KoS)
        idxS = torch.zeros((sS.Hkv, nkeep), dtype=torch.int32, device="cuda")
        if call == "stacked":
            KS, VS, QS = torch.cat(Ks, 0), torch.cat(Vs, 0), torch.cat(Qs, 0)
            KwS = torch.cat(Kws, 0) if args.windowed else None
            wsS = jq.new_workspace(sS)

            def step():
                if args.windowed:
                    jq.evict_layer_windowed(KS, VS, QS, KwS, sS, KoS, VoS, idxS, wsS, stream=stream)
                else:
                    jq.evict_layer(KS, VS, QS, sS, KoS, VoS, idxS, wsS, stream=stream)
        elif call == "layers":
            wsL = jq.new_layers_workspace(s, layers)

            def step():
                jq.evict_layers(Ks, Vs, Qs, s, KoS, VoS, idxS, wsL, stream=stream)
        else:
            step = step_per_layer

    n0 = jq.launch_count()
    total_ms, per_step, clocks = timer.run(step, args.steps, warmup=max(args.warmup, 3))
    launches = jq.launch_count() - n0
    assert jq.last_device_status(ws) == jq.JQ_OK, "device status not ok"
    ms = max_over_ranks(total_ms, world)
    t_layer = ms * 1e-3 / (args.steps * layers)
    value = world * tokens_per_layer / t_layer

    per_layer_calls = host_us = None
    if one_call:
        one_ws = wsR if ragged else (wsL if call == "layers" else wsS)
        assert jq.last_device_status(one_ws) == jq.JQ_OK, "device status not ok"
        # the same work as one call per layer, for comparison (and its results must be the same bits)
        n_pl = max(args.steps // 4, 3)
        tot_pl, _, _ = timer.run(step_per_layer, n_pl)
        if ragged:
            last = rows - wl.Hkv * nkeep
            same = torch.equal(idx.reshape(-1), idxR[last:]) and torch.equal(Ko.reshape(-1, wl.d), KoR[last:])
        else:
            same = torch.equal(idx, idxS[(layers - 1) * wl.Hkv:]) and torch.equal(Ko, KoS[(layers - 1) * wl.Hkv:])
        assert same, "the one-call path and the per-layer calls disagree"
        per_layer_calls = {"ms_per_layer": tot_pl / n_pl / layers, "value": world * wl.L / (tot_pl * 1e-3 / n_pl / layers), "unit": UNIT,
                           "workload": wl.name}
        # host time of a call: calls issued back to back into an empty stream, no synchronisation in between
        host_us = {}
        for name, fn, n in (("jq_evict_layer", lambda: jq.evict_layer(Ks[0], Vs[0], Qs[0], s, Ko, Vo, idx, ws, stream=stream), 16), (CALLS and ("jq_evict_ragged" if ragged else "jq_evict_layers" if call == "layers" else "jq_evict_layer (stacked)"), step, 3)):
            fn(); torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(n):
                fn()
            host_us[name] = (time.perf_counter() - t0) / n * 1e6
            torch.cuda.synchronize()

    # per-stage times through the stage entry points.  The scoring stage runs as many launches as the timed region
    # scored, so that it is measured in the regime the timed region ran in (the SM clock comes down over the first few
    # hundred milliseconds of scoring); the short stages run for 0.15 s so that the clock sampler sees them.
    stage = {}
    if ragged:
        sT, KT, VT, QT = s, Ks[0], Vs[0], Qs[0]                                  # one layer of the longest sequence
        per_launch, wsT, idxT, KoT, VoT = 1, ws, idx, Ko, Vo
    elif one_call:
        sT = sS
        KT, VT, QT = (KS, VS, QS) if call == "stacked" else (torch.cat(Ks, 0), torch.cat(Vs, 0), torch.cat(Qs, 0))
        per_launch, wsT, idxT, KoT, VoT = layers, (wsS if call == "stacked" else jq.new_workspace(sS)), idxS, KoS, VoS
        if args.windowed:
            KwT = KwS
    else:
        sT, KT, VT, QT = s, Ks[0], Vs[0], Qs[0]
        per_launch, wsT, idxT, KoT, VoT = 1, ws, idx, Ko, Vo
        if args.windowed:
            KwT = Kws[0]
    scoresT = torch.empty((sT.Hkv, wl.L), dtype=torch.float32, device="cuda")
    if args.windowed:
        f_score = lambda: jq.score_windowed(KT, QT, KwT, sT, scoresT, wsT, stream=stream)
    else:
        f_score = lambda: jq.score(KT, QT, sT, scoresT, wsT, stream=stream)
    for name, fn in (("score", f_score), ("select", lambda: jq.select_topk(scoresT, sT, idxT, wsT, stream=stream)),
                     ("compact", lambda: jq.compact_kv(KT, VT, idxT, sT, KoT, VoT, stream=stream))):
        if name == "score":
            tot, per, ck = timer.run(fn, max(1, args.steps * (layers // per_launch)))
        else:
            tot, per, ck = timer.run(fn, 4, min_seconds=0.15)
        m = tot / len(per) / per_launch
        stage[name] = {"ms_per_layer": m, "sm_mhz": ck and ck["sm_mhz"], "kcycles_per_layer": kcycles(m, ck)}
    stage_ms = [stage[k]["ms_per_layer"] for k in ("score", "select", "compact")]
    # the scoring stage twice more: as a short burst (4 calls after 3 warm-up calls: the highest clock), and as a loop
    # of at least 0.4 s (the clock the kernel settles at)
    tot, per, _ = timer.run(f_score, 4)
    score_burst_ms = tot / len(per) / per_launch
    tot, per, ck_sus = timer.run(f_score, 4, min_seconds=0.4)
    score_sustained_ms = tot / len(per) / per_launch

    # the second cache the target names (32K keys, 128 query rows per KV head), in the same run: 32 layers, one call
    secondary = None
    if args.workload == "cfg5" and not args.no_secondary and not args.windowed:
        for t in ("KS", "VS", "QS", "KT", "VT", "QT", "scoresT"):
            locals().pop(t, None)
        KT = VT = QT = scoresT = None
        torch.cuda.empty_cache()
        secondary = one_call_cache(W.CFG3 if not args.budget else W.CFG3.with_budget(args.budget), W.CFG3.layers, 8, rank,
                                   max(args.steps, 20), min_seconds=0.3)

    # the CUDA-core comparator of the scoring step (optional, outside the metric): same two passes with fp32 FMAs
    fma_cmp = None
    if args.fma_compare:
        sc1 = torch.empty((wl.Hkv, wl.L), dtype=torch.float32, device="cuda")
        t_tc = timer.run(lambda: jq.score(Ks[0], Qs[0], s, sc1, ws, stream=stream), 8)[0] / 8
        t_fma = timer.run(lambda: jq.score(Ks[0], Qs[0], s, sc1, ws, fma=True, stream=stream), 8)[0] / 8
        fma_cmp = {"what": "jq_score (tcgen05) against jq_score_fma (CUDA cores), one layer per call",
                   "ms_per_layer_tensor": float(t_tc), "ms_per_layer_fma": float(t_fma), "ratio": float(t_fma / t_tc)}

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            peak, peak_src = float(json.load(f)["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"

    # the step after the pass (optional, outside the metric): one decoding position over the pruned cache of a layer
    decode = None
    if args.decode:
        qd = Qs[0][:, -1, :].contiguous()                       # [Hq, d]: the last soft token's queries as a decoding step
        od = torch.empty((wl.Hq, wl.d), dtype=torch.float32, device="cuda")
        wsd = torch.empty(jq.decode_workspace_bytes(wl.Hkv, wl.Hq, nkeep), dtype=torch.uint8, device="cuda")
        # 32 calls captured into a CUDA graph and replayed: a call this short is otherwise timed at the rate the host
        # can issue it
        jq.decode_attention(Ko, Vo, qd, od, wsd, stream=stream)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(32):
                jq.decode_attention(Ko, Vo, qd, od, wsd, stream=torch.cuda.current_stream())
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(4):
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        t_dec = g0.elapsed_time(g1) / (4 * 32)
        dec_bytes = 2.0 * wl.Hkv * nkeep * wl.d * 2
        decode = {"what": "jq_decode_attention over one layer's pruned cache (1 launch)", "n": nkeep, "ms_per_layer": float(t_dec),
                  "roofline": {"bound": "hbm", "kernel": "decode_step", "achieved": dec_bytes / (t_dec * 1e-3) / 1e9, "peak": peak,
                               "peak_source": peak_src, "unit": "GB/s", "frac": dec_bytes / (t_dec * 1e-3) / 1e9 / peak,
                               "bytes_per_launch": dec_bytes, "traffic": None}}

    # end to end through the host-buffer entry point: pinned host tensors in, pinned host results out
    e2e = None
    if not args.no_e2e:
        pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
        hK, hV, hQ = (pin(a) for a in host0)
        hKo = torch.zeros((wl.Hkv, nkeep, wl.d), dtype=torch.int16).pin_memory()
        hVo = torch.zeros_like(hKo).pin_memory()
        hidx = torch.zeros((wl.Hkv, nkeep), dtype=torch.int32).pin_memory()
        buf = torch.empty(jq.host_call_bytes(s), dtype=torch.uint8, device="cuda")
        e2e_layers = 2

        def step_e2e():
            for _ in range(e2e_layers):
                jq.evict_layer_host(hK, hV, hQ, s, hKo, hVo, hidx, buf, stream=stream)
        n_e2e = max(3, min(args.steps, 10))
        tot, _, _ = timer.run(step_e2e, n_e2e, warmup=2)
        t_e2e_layer = max_over_ranks(tot, world) * 1e-3 / (n_e2e * e2e_layers)
        # K and the queries are copied whole; of V (page-locked) only the kept rows cross, read in place by the kernel
        h2d = e2e_layers * (hK.numel() + hQ.numel() + hVo.numel()) * 2
        d2h = e2e_layers * (2 * hKo.numel() * 2 + hidx.numel() * 4)
        e2e = {"value": world * wl.L / t_e2e_layer, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "layers_per_step": e2e_layers, "ms_per_layer": t_e2e_layer * 1e3, "workload": wl.name}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # dominant kernel: score_fused (jq_score, both passes); algorithmic bytes = two reads of K.  One launch
    # covers one layer, or all stacked layers of the step.
    score_bytes = 2 * wl.Hkv * wl.L * wl.d * 2 * per_launch
    ms_launch = float(stage_ms[0]) * per_launch
    achieved = score_bytes / (ms_launch * 1e-3) / 1e9
    layer_gbs = bytes_per_layer / t_layer / 1e9
    traffic_one_layer = NCU_DRAM_BYTES_PER_LAYER.get(wl.name)
    n_exp = 2.0 * wl.R * wl.L * wl.Hkv * per_launch                      # exponentials per launch
    ex2_peak = 148 * 16 * SM_MAX_MHZ * 1e6 / 1e9                         # G/s: 16 results per clock per SM at the maximum SM clock
    step_kc = kcycles(ms / args.steps / layers, clocks)
    # cycles of the scoring stage from its long loop: the clock sampler lags a loop shorter than a few hundred milliseconds
    stage_kc = [kcycles(score_sustained_ms, ck_sus), stage["select"]["kcycles_per_layer"]]
    roofline = {"bound": "hbm", "kernel": "score_fused (jq_score, pass 1 + pass 2)", "achieved": achieved, "peak": peak,
                "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None if traffic_one_layer is None else traffic_one_layer * per_launch,
                "bytes_per_launch": score_bytes, "ms_per_launch": ms_launch,
                "layer_formula_gbs": layer_gbs, "layer_frac_of_peak": layer_gbs / peak,
                "layer_frac_of_8tbs": layer_gbs / 8000.0,
                "ex2_unit": {"note": "the unit that binds this kernel (DRAM is below a quarter of its peak under ncu)",
                             "achieved": n_exp / (ms_launch * 1e-3) / 1e9, "peak": ex2_peak, "unit": "Gexp/s",
                             "frac": n_exp / (ms_launch * 1e-3) / 1e9 / ex2_peak},
                "burst": {"what": "the same kernel timed as a burst of 4 launches (the highest SM clock)",
                          "ms_per_launch": float(score_burst_ms) * per_launch, "achieved": score_bytes / (score_burst_ms * per_launch * 1e-3) / 1e9,
                          "frac": score_bytes / (score_burst_ms * per_launch * 1e-3) / 1e9 / peak},
                "sustained": {"what": "the same kernel timed in a loop of at least 0.4 s (the SM clock it settles at)",
                              "ms_per_launch": float(score_sustained_ms) * per_launch, "achieved": score_bytes / (score_sustained_ms * per_launch * 1e-3) / 1e9,
                              "frac": score_bytes / (score_sustained_ms * per_launch * 1e-3) / 1e9 / peak,
                              "sm_mhz": ck_sus and ck_sus["sm_mhz"], "kcycles_per_layer": kcycles(score_sustained_ms, ck_sus)},
                "stage_ms_per_layer": {k: float(stage[k]["ms_per_layer"]) for k in stage},
                "stages": stage,
                "clock_normalised": {"what": "thousands of SM cycles per layer = time x SM MHz sampled while that loop ran (score: the loop of roofline.sustained)",
                                     "step": step_kc, "score": stage_kc[0], "select": stage_kc[1],
                                     "stages_over_step": None if None in (step_kc, stage_kc[0], stage_kc[1]) or ragged else (stage_kc[0] + stage_kc[1]) / step_kc}}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "ms_per_step_median": float(np.median(per_step)),
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": dict(config_of(wl, layers, distinct, call),
                           softmax=("prefix keys and the causal window keys" if args.windowed else "prefix keys only")),
            "ms_per_layer": t_layer * 1e3, "ms_per_layer_median": float(np.median(per_step)) / layers,
            "per_layer_calls": per_layer_calls, "host_us_per_call": host_us,
            "tokens_discarded_per_s": world * (tokens_per_layer - (sum(w.nkeep for w in seqs) if ragged else nkeep)) / t_layer,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "secondary": secondary}
    if ragged:
        line["config"].update(workload="cfg4-mistral7b-ragged-batch", L=[w.L for w in seqs], sequences=len(seqs),
                              tokens_per_layer=tokens_per_layer, units_per_call=len(RK),
                              l2="inputs larger than L2 (K of one step: %.0f MiB)" % (layers * tokens_per_layer * wl.Hkv * wl.d * 2 / 2**20),
                              note="stage times, per-layer calls and e2e are those of the longest sequence (L = %d)" % wl.L)
    if decode is not None:
        line["decode_step"] = decode
    if fma_cmp is not None:
        line["fma_comparator"] = fma_cmp
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(wl, *host0)
    if world > 1:
        dist.destroy_process_group()
    print(json.dumps(line))


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
