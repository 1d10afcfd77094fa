"""Benchmark of the per-layer KV-cache eviction pass (prefix tokens evicted per second per layer).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg4|cfg3|cfg2] [--budget B]
    python bench.py --impl reference ...      # the fp64 CPU oracle, timed on the host cores

One step = one pass of the whole hot path (scores -> pool -> top-k -> gather) over every layer of
one synthetic cache, on one stream.  Every (layer, KV head) is an independent unit of the pass, so the
layers of a cache are evicted by ONE jq_evict_layer call on tensors that stack the layers along the
KV-head axis (`--call stacked`, the default: K, V [layers*Hkv, L, d], Qwin [layers*Hq, w, d]); the same
work as `layers` separate calls (`--call per-layer`) is also timed and reported.  Prints ONE JSON line.
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
# dram__bytes_read.sum + dram__bytes_write.sum of one score_fused launch on one layer (ncu, see profiles/)
NCU_DRAM_BYTES_PER_LAYER = {"cfg5-llama8b-128k": 355.6e6, "cfg3-llama8b-32k-32layers": 68.8e6}
UNIT = "tokens/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--fma-compare", action="store_true", help="also time the CUDA-core comparator of the scoring step")
    ap.add_argument("--decode", action="store_true", help="also time one decoding step over a layer's pruned cache")
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=["cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--seq", type=int, default=1, help="cfg4 only: which sequence of the ragged batch (0..3)")
    ap.add_argument("--budget", type=int, default=None)
    ap.add_argument("--layers", type=int, default=None, help="layer calls per step (default: the workload's)")
    ap.add_argument("--call", default="layers", choices=["layers", "stacked", "per-layer"],
                    help="layers: one jq_evict_layers call per step on per-layer buffers (default); stacked: one jq_evict_layer call on "
                         "layers concatenated along the KV-head axis; per-layer: one jq_evict_layer call per layer")
    ap.add_argument("--windowed", action="store_true",
                    help="window-inclusive scoring (jq_evict_layer_windowed): the causal keys of the query positions join the softmax")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def pick_workload(args):
    wl = {"cfg2": W.CFG2, "cfg3": W.CFG3, "cfg4": W.CFG4[args.seq % 4], "cfg5": W.CFG5}[args.workload]
    if args.workload == "cfg2":
        wl = W.Workload(wl.name, 2, wl.Hkv, wl.Hq, wl.L, wl.w, wl.budget, layers=32, distinct_layers=32)
    if args.budget:
        wl = wl.with_budget(args.budget)
    return wl


def config_of(wl, layers, distinct, call="per-layer"):
    return {"workload": wl.name, "L": wl.L, "Hkv": wl.Hkv, "Hq": wl.Hq, "d": wl.d, "w": wl.w,
            "budget": wl.budget, "pool": wl.pool, "layers_per_step": layers, "distinct_layers": distinct,
            "call": {"stacked": "one jq_evict_layer call per step, the layers stacked along the KV-head axis",
                     "layers": "one jq_evict_layers call per step, every layer in buffers of its own",
                     "per-layer": "one jq_evict_layer call per layer",
                     "oracle": "the CPU oracle on a bounded sample of one layer"}[call],
            "l2": "inputs larger than L2 (K of one step: %.0f MiB)" % (distinct * wl.Hkv * wl.L * wl.d * 2 / 2**20)}


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
                                       "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.f,
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

    wl = pick_workload(args)
    layers = args.layers or wl.layers
    distinct = min(wl.distinct_layers, layers)
    s = jq.shape(wl.Hkv, wl.Hq, wl.L, wl.w, wl.budget, wl.pool, wl.d)
    nkeep = wl.nkeep

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    host0 = None
    Ks, Vs, Qs, Kws = [], [], [], []
    for i in range(distinct):
        K, V, Q, _ = W.make_layer(wl, layer=i, seq=rank)
        if i == 0:
            host0 = (K, V, Q)
        Ks.append(dev(K)); Vs.append(dev(V)); Qs.append(dev(Q))
        if args.windowed:
            Kws.append(dev(W.make_window_keys(wl, Q, layer=i, seq=rank)))
    ws = jq.new_workspace(s)
    Ko = torch.zeros((wl.Hkv, nkeep, wl.d), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.zeros((wl.Hkv, nkeep), dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def step_per_layer():
        for i in range(layers):
            j = i % distinct
            if args.windowed:
                jq.evict_layer_windowed(Ks[j], Vs[j], Qs[j], Kws[j], s, Ko, Vo, idx, ws, stream=stream)
            else:
                jq.evict_layer(Ks[j], Vs[j], Qs[j], s, Ko, Vo, idx, ws, stream=stream)

    # the layers of the cache stacked along the KV-head axis (a layer repeated in the workload is copied, so
    # that every layer of the step has memory of its own)
    sS = jq.shape(wl.Hkv * layers, wl.Hq * layers, wl.L, wl.w, wl.budget, wl.pool, wl.d)
    if args.windowed and args.call == "layers":
        args.call = "stacked"          # the window-inclusive entry point takes one (stacked) tensor per operand
    one_call = args.call in ("stacked", "layers")
    if one_call:
        order = [i % distinct for i in range(layers)]
        KS = torch.cat([Ks[j] for j in order], 0)
        VS = torch.cat([Vs[j] for j in order], 0)
        QS = torch.cat([Qs[j] for j in order], 0)
        KwS = torch.cat([Kws[j] for j in order], 0) if args.windowed else None
        wsS = jq.new_workspace(sS)
        KoS = torch.zeros((sS.Hkv, nkeep, wl.d), dtype=torch.bfloat16, device="cuda")
        VoS = torch.zeros_like(KoS)
        idxS = torch.zeros((sS.Hkv, nkeep), dtype=torch.int32, device="cuda")

    def step_stacked():
        if args.windowed:
            jq.evict_layer_windowed(KS, VS, QS, KwS, sS, KoS, VoS, idxS, wsS, stream=stream)
        else:
            jq.evict_layer(KS, VS, QS, sS, KoS, VoS, idxS, wsS, stream=stream)

    if args.call == "layers":
        # the layers as a cache holds them: a tensor each (a layer the workload repeats gets a copy of its own)
        seen = set()
        KL, VL, QL = [], [], []
        for j in order:
            KL.append(Ks[j] if j not in seen else Ks[j].clone())
            VL.append(Vs[j] if j not in seen else Vs[j].clone())
            QL.append(Qs[j] if j not in seen else Qs[j].clone())
            seen.add(j)
        wsL = jq.new_layers_workspace(s, layers)

    def step_layers():
        jq.evict_layers(KL, VL, QL, s, KoS, VoS, idxS, wsL, stream=stream)

    step = {"stacked": step_stacked, "layers": step_layers, "per-layer": step_per_layer}[args.call]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    n0 = jq.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = jq.launch_count() - n0
    assert jq.last_device_status(ws) == jq.JQ_OK, "device status not ok"
    if one_call:
        assert jq.last_device_status(wsL if args.call == "layers" else wsS) == jq.JQ_OK, "device status not ok"
        # the same work as one call per layer, for comparison (and its results must be the same bits)
        for _ in range(3):
            step_per_layer()
        barrier()
        e0.record(stream)
        for _ in range(max(args.steps // 4, 3)):
            step_per_layer()
        e1.record(stream)
        barrier()
        ms_pl = e0.elapsed_time(e1) / max(args.steps // 4, 3)
        jlast = (layers - 1) % distinct
        assert torch.equal(idx, idxS[(layers - 1) * wl.Hkv:]) and torch.equal(Ko, KoS[(layers - 1) * wl.Hkv:]), \
            "stacked call and per-layer call disagree"
        per_layer_calls = {"ms_per_layer": ms_pl / layers, "value": world * wl.L / (ms_pl * 1e-3 / layers), "unit": UNIT}
    else:
        per_layer_calls = None

    # per-stage times through the stage entry points: batches of back-to-back calls between events on the
    # launching stream, so that host launch latency is not counted as device time
    scores = [torch.empty((wl.Hkv, wl.L), dtype=torch.float32, device="cuda") for _ in range(min(distinct, 4))]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    nb = max(distinct, 8)
    stage_ms = np.zeros(3)

    def timed(fn):
        for j in range(3):
            fn(j % distinct)
        torch.cuda.synchronize()
        ev[0].record(stream)
        for j in range(nb):
            fn(j % distinct)
        ev[1].record(stream)
        torch.cuda.synchronize()
        return ev[0].elapsed_time(ev[1]) / nb

    if one_call:
        scoresS = torch.empty((sS.Hkv, wl.L), dtype=torch.float32, device="cuda")
        nb = 4
        if args.windowed:
            stage_ms[0] = timed(lambda j: jq.score_windowed(KS, QS, KwS, sS, scoresS, wsS, stream=stream)) / layers
        else:
            stage_ms[0] = timed(lambda j: jq.score(KS, QS, sS, scoresS, wsS, stream=stream)) / layers
        stage_ms[1] = timed(lambda j: jq.select_topk(scoresS, sS, idxS, wsS, stream=stream)) / layers
        stage_ms[2] = timed(lambda j: jq.compact_kv(KS, VS, idxS, sS, KoS, VoS, stream=stream)) / layers
    else:
        if args.windowed:
            stage_ms[0] = timed(lambda j: jq.score_windowed(Ks[j], Qs[j], Kws[j], s, scores[j % len(scores)], ws, stream=stream))
        else:
            stage_ms[0] = timed(lambda j: jq.score(Ks[j], Qs[j], s, scores[j % len(scores)], ws, stream=stream))
        stage_ms[1] = timed(lambda j: jq.select_topk(scores[j % len(scores)], s, idx, ws, stream=stream))
        stage_ms[2] = timed(lambda j: jq.compact_kv(Ks[j], Vs[j], idx, s, Ko, Vo, stream=stream))
    clocks = sampler.stop() if sampler else None

    ms = max_over_ranks(ms, world)
    t_layer = ms * 1e-3 / (args.steps * layers)
    value = job_value(wl, world, t_layer)

    # the CUDA-core comparator of the scoring step (optional, outside the metric): same two passes with fp32 FMAs
    fma_cmp = None
    if args.fma_compare:
        nb = 8
        t_tc = timed(lambda j: jq.score(Ks[j], Qs[j], s, scores[j % len(scores)], ws, stream=stream))
        t_fma = timed(lambda j: jq.score(Ks[j], Qs[j], s, scores[j % len(scores)], ws, fma=True, stream=stream))
        fma_cmp = {"what": "jq_score (tcgen05) against jq_score_fma (CUDA cores), one layer per call",
                   "ms_per_layer_tensor": float(t_tc), "ms_per_layer_fma": float(t_fma), "ratio": float(t_fma / t_tc)}

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
        decode = {"what": "jq_decode_attention over one layer's pruned cache (1 launch)", "n": nkeep, "ms_per_layer": float(t_dec),
                  "cache_gbs": 2.0 * wl.Hkv * nkeep * wl.d * 2 / (t_dec * 1e-3) / 1e9}

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
        n_e2e = max(3, min(args.steps, 10))
        for _ in range(2):
            jq.evict_layer_host(hK, hV, hQ, s, hKo, hVo, hidx, buf, stream=stream)
        barrier()
        e0.record(stream)
        for _ in range(n_e2e * e2e_layers):
            jq.evict_layer_host(hK, hV, hQ, s, hKo, hVo, hidx, buf, stream=stream)
        e1.record(stream)
        barrier()
        t_e2e_layer = max_over_ranks(e0.elapsed_time(e1), world) * 1e-3 / (n_e2e * e2e_layers)
        # K and the queries are copied whole; of V (page-locked) only the kept rows cross, read in place by the kernel
        h2d = e2e_layers * (hK.numel() + hQ.numel() + hVo.numel()) * 2
        d2h = e2e_layers * (2 * hKo.numel() * 2 + hidx.numel() * 4)
        e2e = {"value": world * wl.L / t_e2e_layer, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "layers_per_step": e2e_layers, "ms_per_layer": t_e2e_layer * 1e3}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            peak, peak_src = float(json.load(f)["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    # dominant kernel: score_fused (jq_score, both passes); algorithmic bytes = two reads of K.  One launch
    # covers one layer, or all stacked layers of the step.
    per_launch = layers if one_call else 1
    score_bytes = 2 * wl.Hkv * wl.L * wl.d * 2 * per_launch
    ms_launch = float(stage_ms[0]) * per_launch
    achieved = score_bytes / (ms_launch * 1e-3) / 1e9
    layer_gbs = W.formula_bytes(wl) / t_layer / 1e9
    # DRAM bytes of one score_fused launch on ONE layer of this workload from an ncu capture of the kernel
    # as it stands (profiles/), scaled to the launch by the layers it covers; None where no capture exists
    traffic_one_layer = NCU_DRAM_BYTES_PER_LAYER.get(wl.name)
    n_exp = 2.0 * wl.R * wl.L * wl.Hkv * per_launch                      # exponentials per launch
    ex2_peak = 148 * 16 * 1965e6 / 1e9                                   # G/s: 16 results per clock per SM at the maximum SM clock
    roofline = {"bound": "hbm", "kernel": "score_fused (jq_score, pass 1 + pass 2)", "achieved": achieved, "peak": peak,
                "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None if traffic_one_layer is None else traffic_one_layer * per_launch,
                "bytes_per_launch": score_bytes, "ms_per_launch": ms_launch,
                "layer_formula_gbs": layer_gbs, "layer_frac_of_peak": layer_gbs / peak,
                "layer_frac_of_8tbs": layer_gbs / 8000.0,
                "ex2_unit": {"note": "the unit that binds this kernel (DRAM is below a quarter of its peak under ncu)",
                             "achieved": n_exp / (ms_launch * 1e-3) / 1e9, "peak": ex2_peak, "unit": "Gexp/s",
                             "frac": n_exp / (ms_launch * 1e-3) / 1e9 / ex2_peak},
                "stage_ms_per_layer": {"score": float(stage_ms[0]), "select": float(stage_ms[1]), "compact": float(stage_ms[2])}}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": dict(config_of(wl, layers, distinct, args.call),
                           softmax=("prefix keys and the causal window keys" if args.windowed else "prefix keys only")),
            "ms_per_layer": t_layer * 1e3,
            "per_layer_calls": per_layer_calls,
            "tokens_discarded_per_s": world * (wl.L - nkeep) / t_layer,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline}
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
