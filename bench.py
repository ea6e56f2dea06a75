#!/usr/bin/env python
"""Benchmark of the MoE layer decode step at batch 1 on the 35B-class layer shape.

One "step" is one layer-step: the prerouter head scores the next step's experts from this step's
hidden state (logits, softmax, top-k, renormalised gates), the routing predicted one step earlier
is mapped through the slot table, the K int4 SwiGLU experts with their unmerged LoRA delta run
over those slots, and the K outputs are reduced by their gate weights -- all through the C-ABI
call ``moe_layer_decode``.

Default arm (``--impl b200``):
  value : layer-steps per second with everything resident in HBM.  The workload rotates over
          several independently seeded instances of the layer (each with all E experts resident),
          so the bytes a step streams are far outside the L2 and come from HBM.  Steps depend on
          one another through the routing only (step t+1 consumes the top-k that step t produced;
          the hidden states are independent draws, as the configuration states) and are launched
          from CUDA graphs.  Whatever ``--steps`` says, the timed region is WINDOWS windows of
          WINDOW_STEPS steps each, timed with CUDA events on the launching stream; the median
          window is reported (``config.timed_steps`` / ``config.windows``), so the number does not
          depend on the flag.
  dependent : the same layer-steps when the hidden state of step t+1 is produced on the device from
          step t's output, x(t+1) = bf16(rmsnorm(x(t) + y(t))): no step can start its arithmetic
          before the previous one has finished -- the latency a decoder sees.
  e2e   : the same metric with HOST buffers: the experts live in a pinned-host store, the HBM pool
          has the configuration's 8 slots, every step copies its hidden state host->device, stages
          the missing experts with cudaMemcpyAsync, runs the layer-step and reads y back.
  secondary : batched decode (cfg4 shape) and prefill (cfg5 shape) on the same resident layer.
  roofline / cpu_baseline / clocks: see the keys of the JSON line.
Reference arm (``--impl reference``): the fp64 CPU oracle, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import synth  # noqa: E402

METRIC = "moe_layer_decode_tok_per_s_batch1"
UNIT = "tok/s"
WORKLOAD = "cfg2: one 35B-class MoE layer (H2048 I512 E256 top-8 int4 g64 LoRA r16), batch-1 decode"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from an ncu
# capture of this workload (not measured by this run: reported as "from profile").
NCU_TRAFFIC_BYTES = 15_621_120
WINDOWS = 5            # timed windows; the median is reported
WINDOW_STEPS = 2560    # layer-steps per window: one replay of a 2560-step graph


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the GPU is under load."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        self.period = period_s
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
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "sw_power_cap": 0x4, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------ workload

def _physical_device(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def build_instances(edg, layer_io, cfg, desc, n_inst, first_layer):
    """Pinned host layers for `n_inst` independently seeded instances of the layer."""
    R = edg.record_bytes(desc)
    import torch
    hosts = [torch.empty((cfg.E, R), dtype=torch.uint8, pin_memory=True) for _ in range(n_inst)]

    def fill(job):
        i, e = job
        edg.pack_expert(desc, synth.expert_tensors(cfg, first_layer + i, e), hosts[i].numpy()[e])

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        list(ex.map(fill, [(i, e) for i in range(n_inst) for e in range(cfg.E)]))
    return hosts


def run_b200(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local_rank = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    from paper_2609_18063_b200 import build
    build.build()
    import paper_2609_18063_b200 as edg
    from paper_2609_18063_b200 import layer_io

    cfg = synth.CONFIGS["cfg2"]
    n_inst = args.instances
    from paper_2609_18063_b200 import replicas
    first_layer = replicas.first_instance(rank, n_inst)   # replicas: every rank serves its own layer instances
    desc = edg.make_desc(cfg, n_slots=cfg.E, out_dtype="f32")
    R = edg.record_bytes(desc)
    K, E, H = cfg.K, cfg.E, cfg.H

    hosts = build_instances(edg, layer_io, cfg, desc, n_inst, first_layer)
    loras, keep = [], []
    for i in range(n_inst):
        lo, k = layer_io.lora_to_device(desc, [synth.lora_tensors(cfg, first_layer + i, 0)])
        loras.append(lo); keep.append(k)
    W = torch.from_numpy(np.stack([synth.prerouter_weights(cfg, first_layer + i) for i in range(n_inst)])).cuda()

    # ---- resident arm: all experts of all instances in HBM, slot e of instance i holds expert e
    pool = torch.empty((n_inst, E, R), dtype=torch.uint8, device="cuda")
    tables = torch.empty((n_inst, E), dtype=torch.int32, device="cuda")
    copy_stream = torch.cuda.Stream()
    store = edg.Store(desc, hosts, pool, tables, loras, copy_stream)
    for i in range(n_inst):
        for e0 in range(0, E, 64):
            edg.stage_experts_to_slots(store, i, np.arange(e0, min(E, e0 + 64), dtype=np.int32))
    copy_stream.synchronize()
    assert store.stats()["misses"] == n_inst * E

    NX = 256
    X_bits = synth.hidden_states(cfg, NX, layer=first_layer, stream=100)
    xd = layer_io.bits_to_device(X_bits, torch.bfloat16)
    y = torch.zeros((NX, H), dtype=torch.float32, device="cuda")
    inds = torch.zeros((2, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((2, K), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(desc)

    def step(s):
        i = s % n_inst
        edg.moe_layer_decode(store, i, xd[s % NX], inds[s % 2], gates[s % 2], W[(s + 1) % n_inst],
                             inds[(s + 1) % 2], gates[(s + 1) % 2], None, y[s % NX], ws)

    # routing of step 0 comes from a "last prompt token" state
    edg.prerouter_topk(desc, W[0], xd[NX - 1], 1, inds[0], gates[0], None)
    torch.cuda.synchronize()

    G = WINDOW_STEPS                       # steps per CUDA graph: a window is one replay
    G_DEP = 256                            # the dependent arms: nothing overlaps across steps, so the graph size is immaterial
    if NX % n_inst or n_inst % 2 and n_inst != 1:
        raise SystemExit("--instances must be even (or 1) and divide 256")
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())

    # touch every instance once outside capture (an even count keeps the two-entry routing ring in
    # phase), so that no staging event is waited on inside a graph
    with torch.cuda.stream(stream):
        for s in range(2 * n_inst):
            step(s)
        stream.synchronize()

    def capture(n_steps, base=0):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g, stream=stream):
                for s in range(base, base + n_steps):
                    step(s)
        return g

    steps, warmup = args.steps, max(args.warmup, 3)
    # The hand-off ring has 128 slots and a captured chain has its slots baked in, so a graph that is
    # replayed again and again holds a multiple of 128 steps.  A replay is stream-ordered behind the
    # one before it, so the chain drains and refills once per replay (about half the lifetime of a
    # CTA, 0.1 ms): the graph holds a whole window of 2560 steps (64 tokens x 40 layers' worth), not 256.
    store.set_chaining(1)                  # opt in: the captured steps are chained through the routing
    g_full = capture(G)
    reps = WINDOW_STEPS // G

    def timed_windows(graph, reps=reps):
        """WINDOWS windows of `reps` replays each, one event pair per window; ms per window, max over ranks."""
        out = []
        with torch.cuda.stream(stream):
            for _ in range(WINDOWS):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(reps):
                    graph.replay()
                e1.record(stream)
                out.append((e0, e1))
            stream.synchronize()
        return [replicas.max_over_ranks(a.elapsed_time(b), "cuda") for a, b in out]

    sampler = ClockSampler(_physical_device(local_rank))
    with torch.cuda.stream(stream):
        for _ in range(max(2, (warmup + G - 1) // G)):
            g_full.replay()
        stream.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    window_ms = timed_windows(g_full)
    with torch.cuda.stream(stream):
        # keep the GPU under the same load a little longer so the clock sampler sees it
        t_end = time.time() + 0.3
        while time.time() < t_end:
            g_full.replay()
        stream.synchronize()
    clocks = sampler.stop()
    torch.cuda.synchronize()
    status = edg.workspace_status(ws)
    if status != 0 or not bool(torch.isfinite(y).all()):
        raise SystemExit(f"bench: bad device status {status} or non-finite output")

    ms_med = statistics.median(window_ms)
    value = replicas.whole_job_rate(world, WINDOW_STEPS, ms_med)
    ms_per_step = ms_med / WINDOW_STEPS

    # ---- dependent arm: x(t+1) = bf16(rmsnorm(x(t) + y(t))) on the device, chaining off
    dependent = None
    if not args.no_dependent:
        store.set_chaining(0)
        xdep = torch.zeros((2, H), dtype=torch.bfloat16, device="cuda")
        xdep[0] = xd[0]
        ydep = torch.zeros((H,), dtype=torch.float32, device="cuda")

        def dep_step(s_):
            i = s_ % n_inst
            edg.moe_layer_decode(store, i, xdep[s_ % 2], inds[s_ % 2], gates[s_ % 2], W[(s_ + 1) % n_inst],
                                 inds[(s_ + 1) % 2], gates[(s_ + 1) % 2], None, ydep, ws)
            edg.next_hidden_state(desc, xdep[s_ % 2], ydep, xdep[(s_ + 1) % 2], 1e-6)

        with torch.cuda.stream(stream):
            for s_ in range(2 * n_inst):
                dep_step(s_)
            stream.synchronize()
        g_dep = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g_dep, stream=stream):
                for s_ in range(G_DEP):
                    dep_step(s_)
            g_dep.replay()
            stream.synchronize()
        dep_ms = statistics.median(timed_windows(g_dep, WINDOW_STEPS // G_DEP))
        status = edg.workspace_status(ws)
        if status != 0 or not bool(torch.isfinite(ydep).all()) or not bool(torch.isfinite(xdep.float()).all()):
            raise SystemExit(f"bench: dependent arm: bad device status {status} or non-finite state")
        dep_step_ms = dep_ms / WINDOW_STEPS
        # the same chain with the next state written by the layer kernel itself and the steps chained:
        # step t+1 is resident, routed and has its first weights when x(t+1) is written
        store.set_chaining(1)

        def dep2_step(s_):
            i = s_ % n_inst
            edg.moe_layer_decode_dependent(store, i, xdep[s_ % 2], inds[s_ % 2], gates[s_ % 2], W[(s_ + 1) % n_inst],
                                           inds[(s_ + 1) % 2], gates[(s_ + 1) % 2], None, ydep, xdep[(s_ + 1) % 2], ws, 1e-6)

        with torch.cuda.stream(stream):
            for s_ in range(2 * n_inst):
                dep2_step(s_)
            stream.synchronize()
        g_dep2 = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(g_dep2, stream=stream):
                for s_ in range(G_DEP):
                    dep2_step(s_)
            g_dep2.replay()
            stream.synchronize()
        dep2_ms = statistics.median(timed_windows(g_dep2, WINDOW_STEPS // G_DEP))
        status = edg.workspace_status(ws)
        if status != 0 or not bool(torch.isfinite(ydep).all()) or not bool(torch.isfinite(xdep.float()).all()):
            raise SystemExit(f"bench: fused dependent arm: bad device status {status} or non-finite state")
        store.set_chaining(0)
        dep2_step_ms = dep2_ms / WINDOW_STEPS
        dependent = {"value": round(replicas.whole_job_rate(world, WINDOW_STEPS, dep2_ms), 1), "unit": UNIT,
                     "ms_per_step": round(dep2_step_ms, 6),
                     "hbm_gbs_on_expert_bytes": round(K * R / (dep2_step_ms * 1e-3) / 1e9, 1),
                     "frac_of_peak": round(K * R / (dep2_step_ms * 1e-3) / 1e9 / _peaks()[0], 4),
                     "dependency": "x(t+1) = bf16(rmsnorm(x(t) + y(t))) computed on the device: every step waits for the one before it",
                     "launch": f"moe_layer_decode_dependent: one kernel per step writes y and x(t+1); steps chained (the next step "
                               f"is resident, routed and streaming its first weights while it waits for x); CUDA graphs of {G_DEP} steps",
                     "unchained_two_kernels": {"ms_per_step": round(dep_step_ms, 6),
                                               "value": round(replicas.whole_job_rate(world, WINDOW_STEPS, dep_ms), 1),
                                               "launch": "layer-step + next-state norm as two stream-ordered kernels, chaining off"},
                     "timed_steps": WINDOWS * WINDOW_STEPS, "windows": WINDOWS}

    # ---- batched decode and prefill on the same resident layer (secondary figures)
    secondary = None
    if not args.no_secondary and world == 1:
        secondary = run_secondary(edg, layer_io, cfg, desc, pool[0], loras[0], W[0], R)

    # ---- e2e arm: pinned-host store, 8 slots, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(edg, layer_io, cfg, hosts[0], loras[0], W[0], X_bits, args, world)

    # ---- roofline of the dominant work: the int4 expert bytes one step streams
    peak, how = _peaks()
    alg_bytes = K * R
    launches_per_step = 1                  # one fused kernel: prerouter + take + FFN + reduce
    achieved = alg_bytes / (ms_per_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "traffic": NCU_TRAFFIC_BYTES,
                "traffic_source": "from profile (ncu capture of this kernel and workload), not measured by this run",
                "peak_kind": how + " (burst copy)",
                "kernel": "fused_layer_kernel (one launch per layer-step; duration = timed region / launches)",
                "algorithmic_bytes_per_launch": alg_bytes}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, args.cpu_seconds)

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": round(ms_per_step, 6), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int4 weights, bf16 activations, fp32 accumulate",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "resident_instances": n_inst,
                       "hbm_working_set_bytes": n_inst * E * R,
                       "l2": "inputs larger than L2: steps rotate over the instances, routing iid from the prerouter",
                       "routing": "redrawn every step from the prerouter (step t+1 consumes step t's top-k)",
                       "dependency": "routing only: hidden states are independent draws, so steps overlap on the GPU; see 'dependent' for data-dependent steps",
                       "timed_steps": WINDOWS * WINDOW_STEPS, "windows": WINDOWS,
                       "window_ms": [round(m, 4) for m in window_ms],
                       "timing": f"median of {WINDOWS} windows of {WINDOW_STEPS} steps, whatever --steps says",
                       "launch": f"CUDA graphs of {G} steps, chained (edg_store_set_chaining 1)",
                       "parallelism": "replicas only" if world > 1 else "1 GPU"},
            "clocks": clocks, "e2e": e2e, "dependent": dependent, "secondary": secondary,
            "gpu_launches": launches_per_step * WINDOWS * WINDOW_STEPS,
            "roofline": roofline, "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    store.close()
    if world > 1:
        dist.destroy_process_group()


def _event_ms(fn, iters, warmup=3):
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _graph_ms(fn, per_graph, reps, warm=2):
    """ms per call of fn with `per_graph` calls captured into one CUDA graph and replayed `reps` times."""
    import torch
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for _ in range(per_graph):
                fn()
        for _ in range(warm):
            g.replay()
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(reps):
            g.replay()
        e1.record(st)
        st.synchronize()
    torch.cuda.current_stream().wait_stream(st)
    return e0.elapsed_time(e1) / (reps * per_graph)


def run_secondary(edg, layer_io, cfg, desc, pool, lora, W, R):
    """Batched decode (cfg4 shape: 64 concurrent tokens) and prefill (cfg5 shape: 4096 tokens, Zipf(1.1)
    popularity) on one resident layer of the headline workload (same layer shape; `--workload cfg4` /
    `cfg5` print the full lines on their own seeds)."""
    import torch
    K, E, H, I = cfg.K, cfg.E, cfg.H, cfg.I
    peak_hbm, how = _peaks()
    peak_tf = 1385.0
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        peak_tf = float(json.load(open(pk))["bf16_tflops_sustained"])
    table = torch.arange(E, dtype=torch.int32, device="cuda")
    out = {}
    # ---- cfg4 shape
    c4 = synth.CONFIGS["cfg4"]
    T = c4.T
    X = [layer_io.bits_to_device(synth.hidden_states(c4, T, stream=200 + i), torch.bfloat16) for i in range(4)]
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    y = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(desc, T)
    it, unions = [0], []

    def step4():
        x = X[it[0] % 4]; it[0] += 1
        edg.prerouter_topk_tokens(desc, W, x, T, inds, gates, None)
        edg.moe_expert_ffn_int4_lora(desc, pool, table, T, inds, None, gates, x, lora, y, ws)

    for _ in range(4):
        step4(); torch.cuda.synchronize(); unions.append(len(torch.unique(inds)))
    ms = _graph_ms(step4, 4, 6)          # (the step's eight kernels from a CUDA graph, as `--workload cfg4` does)
    ok = edg.workspace_status(ws) == 0 and bool(torch.isfinite(y).all())
    union = float(np.mean(unions))
    ach = union * R / (ms * 1e-3) / 1e9
    out["cfg4_shape"] = {"tokens": T, "ms_per_step": round(ms, 5), "tok_per_s": round(T / (ms * 1e-3), 1),
                         "experts_touched": union, "hbm_gbs_on_union_bytes": round(ach, 1),
                         "frac_of_hbm_peak": round(ach / peak_hbm, 4), "ok": ok}
    del ws, y
    # ---- cfg5 shape
    c5 = synth.CONFIGS["cfg5"]
    T = c5.T
    x = layer_io.bits_to_device(synth.hidden_states(c5, T, stream=300), torch.bfloat16)
    logits = torch.from_numpy(synth.zipf_router_logits(c5, T)).cuda()
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    y = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(desc, T)

    def step5():
        edg.softmax_topk_rows(desc, logits, T, inds, gates)
        edg.moe_expert_ffn_int4_lora(desc, pool, table, T, inds, None, gates, x, lora, y, ws)

    ms = _event_ms(step5, 10)
    ok = edg.workspace_status(ws) == 0 and bool(torch.isfinite(y).all())
    flops = T * K * (6.0 * H * I + 2.0 * cfg.rank * (2 * H + 3 * I + H))
    tf = flops / (ms * 1e-3) / 1e12
    out["cfg5_shape"] = {"tokens": T, "ms_per_step": round(ms, 4), "tok_per_s": round(T / (ms * 1e-3), 1),
                         "tflops_algorithmic": round(tf, 1), "frac_of_tensor_peak": round(tf / peak_tf, 4),
                         "peak_kind": "measured sustained bf16 GEMM", "ok": ok}
    return out


def run_e2e(edg, layer_io, cfg, host_layer, lora, W, X_bits, args, world):
    """Config 2 as written: pinned-host expert store, 8 slots, one layer; per step the hidden state
    goes host->device, the routed experts that are not resident are staged, the layer-step runs and
    y comes back to the host."""
    import torch
    import torch.distributed as dist
    K, E, H = cfg.K, cfg.E, cfg.H
    desc = edg.make_desc(cfg, n_slots=cfg.n_slots, out_dtype="f32")
    R = edg.record_bytes(desc)
    slots = torch.empty((1, cfg.n_slots, R), dtype=torch.uint8, device="cuda")
    tables = torch.empty((1, E), dtype=torch.int32, device="cuda")
    cs = torch.cuda.Stream()
    store = edg.Store(desc, [host_layer], slots, tables, [lora], cs)
    ws = layer_io.new_workspace(desc)
    NX = X_bits.shape[0]
    x_host = torch.from_numpy(X_bits.view(np.int16).copy()).pin_memory()
    x_dev = torch.empty((H,), dtype=torch.int16, device="cuda")
    y_dev = torch.empty((H,), dtype=torch.float32, device="cuda")
    y_host = torch.empty((H,), dtype=torch.float32).pin_memory()
    inds = torch.zeros((2, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((2, K), dtype=torch.float32, device="cuda")
    # the predicted routing is mirrored into pinned host memory by the kernels: the stager reads it
    # there, without a device-to-host copy
    mirror = torch.full((2, K), -1, dtype=torch.int32).pin_memory()
    mir = mirror.numpy()
    st = torch.cuda.current_stream()
    edg.prerouter_topk(desc, W, layer_io.bits_to_device(X_bits[NX - 1], torch.bfloat16), 1, inds[0], gates[0], None,
                       inds_host_mirror_opt=mirror[0])
    st.synchronize()

    def step(s):
        x_dev.copy_(x_host[s % NX], non_blocking=True)
        cur, nxt = s % 2, (s + 1) % 2
        edg.stage_experts_to_slots(store, 0, mir[cur])             # the prediction made one step earlier
        mir[nxt] = -1
        edg.moe_layer_decode(store, 0, x_dev, inds[cur], gates[cur], W, inds[nxt], gates[nxt],
                             None, y_dev, ws, inds_next_host_mirror_opt=mirror[nxt])
        y_host.copy_(y_dev, non_blocking=True)
        st.synchronize()

    n = max(64, min(args.steps, args.e2e_steps) // 2 * 2)  # an even count: the routing alternates between two buffers
    for s in range(max(4, min(args.warmup, 20) // 2 * 2)):
        step(s)
    base = store.stats()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(n):
        step(s)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    from paper_2609_18063_b200 import replicas
    ms_max = replicas.max_over_ranks(ms, "cuda")
    after = store.stats()
    miss_bytes = (after["bytes_copied"] - base["bytes_copied"]) / n
    table_bytes = (after["table_updates"] - base["table_updates"]) * E * 4 / n
    out = {"value": round(replicas.whole_job_rate(world, n, ms_max), 1), "unit": UNIT,
           "h2d_bytes_per_step": int(H * 2 + miss_bytes + table_bytes), "d2h_bytes_per_step": H * 4 + K * 4,
           "d2h_note": "y by cudaMemcpyAsync; the K predicted indices by the kernel's own stores into mapped pinned memory",
           "steps": n, "slots": cfg.n_slots,
           "misses_per_step": round((after["misses"] - base["misses"]) / n, 3),
           "note": "pinned-host expert store, 8 slots, experts staged on demand by cudaMemcpyAsync: bound by host->device copy bandwidth"}
    store.close()
    return out


# ------------------------------------------------------------------ CPU oracle timing

def _oracle_steps(cfg, n_steps, budget_s):
    """Times the oracle's layer-step on pre-generated inputs; returns (steps done, seconds, threads)."""
    from oracle import moe_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = 1
    W = synth.prerouter_weights(cfg, 0)
    X = synth.hidden_states(cfg, n_steps + 1, stream=100)
    lora = synth.lora_tensors(cfg, 0, 0)
    inds, gates = orc.softmax_topk(orc.prerouter_logits(W, X[n_steps]), cfg.K)
    done, spent = 0, 0.0
    for t in range(n_steps):
        experts = {int(e): synth.expert_tensors(cfg, 0, int(e)) for e in inds}      # input generation: untimed
        t0 = time.perf_counter()
        _, _, _, inds, gates, _ = orc.moe_layer_decode(X[t], inds, gates, W, cfg.K, experts.__getitem__,
                                                       lambda e: lora, cfg.lora_scale, cfg.group)
        spent += time.perf_counter() - t0
        done += 1
        if spent >= budget_s:
            break
    return done, spent, threads


def cpu_baseline(cfg, budget_s):
    done, spent, threads = _oracle_steps(cfg, 1000, budget_s)
    return {"value": round(done / spent, 3), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{done} consecutive layer-steps of the same workload (fp64 numpy oracle, {spent:.1f} s)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if rank != 0:
        return
    cfg = synth.CONFIGS["cfg2"]
    _oracle_steps(cfg, max(1, min(args.warmup, 2)), 5.0)
    done, spent, threads = _oracle_steps(cfg, args.steps, 120.0)
    value = done / spent
    sample = (f"{done} of the {args.steps} requested layer-steps were run (time-bounded sample); "
              "each is one full oracle layer-step")
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(1e3 / value, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "parallelism": "host cores"},
            "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "kind": "oracle", "cores": threads, "sample": sample},
            "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------ secondary workloads (not the headline line)

def _time_steps(fn, steps, warmup, stream_sync):
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def run_cfg4(args):
    """Batched decode: 64 concurrent tokens, independent top-8 from the head, all experts resident."""
    import torch
    from paper_2609_18063_b200 import build
    build.build()
    import paper_2609_18063_b200 as edg
    from paper_2609_18063_b200 import layer_io
    cfg = synth.CONFIGS["cfg4"]
    T, K, E, H = cfg.T, cfg.K, cfg.E, cfg.H
    desc = edg.make_desc(cfg, n_slots=E, out_dtype="f32")
    R = edg.record_bytes(desc)
    host = build_instances(edg, layer_io, cfg, desc, 1, 0)[0]
    pool = host.cuda()
    table = torch.arange(E, dtype=torch.int32, device="cuda")
    lora, keep = layer_io.lora_to_device(desc, [synth.lora_tensors(cfg, 0, 0)])
    W = torch.from_numpy(synth.prerouter_weights(cfg, 0)).cuda()
    NX = 8
    X = [layer_io.bits_to_device(synth.hidden_states(cfg, T, stream=200 + i), torch.bfloat16) for i in range(NX)]
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    y = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(desc, T)
    it = [0]
    unions = []

    def step():
        x = X[it[0] % NX]; it[0] += 1
        edg.prerouter_topk_tokens(desc, W, x, T, inds, gates, None)
        edg.moe_expert_ffn_int4_lora(desc, pool, table, T, inds, None, gates, x, lora, y, ws)

    for i in range(NX):
        step(); torch.cuda.synchronize(); unions.append(len(torch.unique(inds)))
    # the NX steps (eight kernels each) as one CUDA graph, replayed: no launch gaps between the small kernels
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for i in range(NX):
                step()
        reps = max(1, (args.steps + NX - 1) // NX)
        for _ in range(max(1, (max(args.warmup, 3) + NX - 1) // NX)):
            g.replay()
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(reps):
            g.replay()
        e1.record(st)
        st.synchronize()
    ms = e0.elapsed_time(e1) / (reps * NX)
    torch.cuda.current_stream().wait_stream(st)
    assert edg.workspace_status(ws) == 0 and bool(torch.isfinite(y).all())
    peak, how = _peaks()
    union = float(np.mean(unions))
    alg = union * R
    ach = alg / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "moe_layer_batched_decode_tok_per_s", "value": round(T / (ms * 1e-3), 1), "unit": "tok/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms, 5),
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                      "dtype": "int4 weights, fp16 mma operands, fp32 accumulate", "data": "synthetic",
                      "config": {"workload": "cfg4: 64 concurrent tokens, top-8 of 256, int4 g64 + LoRA r16, union pool of 256 slots",
                                 "experts_touched_per_step": union, "l2": "union of routed experts (~390 MB) exceeds the 126 MB L2"},
                      "roofline": {"bound": "hbm", "achieved": round(ach, 1), "peak": peak, "unit": "GB/s", "frac": round(ach / peak, 4),
                                   "traffic": None, "peak_kind": how, "algorithmic_bytes_per_launch": int(alg)},
                      "launch": f"CUDA graph of {NX} steps, replayed {reps} times",
                      "gpu_launches": 8 * reps * NX}))


def run_cfg5(args):
    """Prefill: 4096 tokens, Zipf(1.1) expert popularity, grouped tensor-core path."""
    import torch
    from paper_2609_18063_b200 import build
    build.build()
    import paper_2609_18063_b200 as edg
    from paper_2609_18063_b200 import layer_io
    cfg = synth.CONFIGS["cfg5"]
    T, K, E, H, I = cfg.T, cfg.K, cfg.E, cfg.H, cfg.I
    desc = edg.make_desc(cfg, n_slots=E, out_dtype="f32")
    host = build_instances(edg, layer_io, cfg, desc, 1, 0)[0]
    pool = host.cuda()
    table = torch.arange(E, dtype=torch.int32, device="cuda")
    lora, keep = layer_io.lora_to_device(desc, [synth.lora_tensors(cfg, 0, 0)])
    x = layer_io.bits_to_device(synth.hidden_states(cfg, T, stream=300), torch.bfloat16)
    logits = torch.from_numpy(synth.zipf_router_logits(cfg, T)).cuda()
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    y = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(desc, T)

    def step():
        edg.softmax_topk_rows(desc, logits, T, inds, gates)
        edg.moe_expert_ffn_int4_lora(desc, pool, table, T, inds, None, gates, x, lora, y, ws)

    steps = min(args.steps, 50)
    ms = _time_steps(step, steps, max(min(args.warmup, 5), 3), None)
    assert edg.workspace_status(ws) == 0 and bool(torch.isfinite(y).all())
    flops = T * K * (6.0 * H * I + 2.0 * cfg.rank * (2 * H + 3 * I + H))      # base GEMMs + LoRA
    tf = flops / (ms * 1e-3) / 1e12
    peak = 1385.0
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        peak = float(json.load(open(pk))["bf16_tflops_sustained"])
    print(json.dumps({"metric": "moe_layer_prefill_tok_per_s", "value": round(T / (ms * 1e-3), 1), "unit": "tok/s",
                      "n_gpus": 1, "steps": steps, "warmup": 3, "ms_per_step": round(ms, 4), "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "int4 weights, fp16 mma operands, fp32 accumulate",
                      "data": "synthetic",
                      "config": {"workload": "cfg5: 4096-token prefill, top-8 of 256 with Zipf(1.1) popularity, int4 g64 + LoRA r16"},
                      "roofline": {"bound": "tensor", "achieved": round(tf, 1), "peak": peak, "unit": "TFLOP/s",
                                   "frac": round(tf / peak, 4), "traffic": None,
                                   "peak_kind": "measured sustained bf16 GEMM (fp16 runs at the same rate)"},
                      "gpu_launches": 10 * steps}))


def _h2d_fit(R):
    """Host-to-device copy cost as a + b * bytes (the analogue of the paper's load-cost model, Sec. 5.3):
    batches of 64 copies of 1, 2, 4 and 8 records from pinned memory on one stream, least squares."""
    import torch
    sizes = [R, 2 * R, 4 * R, 8 * R]
    src = torch.empty((8 * R,), dtype=torch.uint8, pin_memory=True)
    dst = torch.empty((64, 8 * R), dtype=torch.uint8, device="cuda")
    per_copy = []
    for n in sizes:
        for rep in range(2):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(64):
                dst[i, :n].copy_(src[:n], non_blocking=True)
            e1.record()
            torch.cuda.synchronize()
        per_copy.append(e0.elapsed_time(e1) / 64 * 1e-3)
    A = np.stack([np.ones(len(sizes)), np.array(sizes, dtype=np.float64)], axis=1)
    (a, b), *_ = np.linalg.lstsq(A, np.array(per_copy), rcond=None)
    return {"a_us_per_copy": round(a * 1e6, 2), "b_us_per_MB": round(b * 1e12, 2), "GBps_asymptotic": round(1e-9 / b, 1),
            "us_per_record_copy": round(per_copy[0] * 1e6, 1)}


def run_cfg3(args):
    """The 40-layer expert stack: prediction-driven staging from the pinned-host store (18.1 GB of
    records), 512 tokens per arm; arms over pool size, staging policy and routing statistics."""
    import torch
    from paper_2609_18063_b200 import build
    build.build()
    import paper_2609_18063_b200 as edg
    from paper_2609_18063_b200 import layer_io
    from paper_2609_18063_b200.decoder import StackDecoder
    cfg = synth.CONFIGS["cfg3"]
    L, K, E, H = cfg.n_layers, cfg.K, cfg.E, cfg.H
    desc0 = edg.make_desc(cfg)
    R = edg.record_bytes(desc0)
    tokens = max(8, min(args.steps, 512))
    warm = 8
    # ---- the pinned-host tier: one 453 MB allocation per layer; alias only where pinning is refused
    hosts, refusal = [], None
    for l in range(L):
        try:
            hosts.append(torch.empty((E, R), dtype=torch.uint8, pin_memory=True))
        except RuntimeError as ex:                      # keep the refusal text, alias the rest
            refusal = f"layer {l}: {str(ex).splitlines()[0][:160]}"
            break
    n_distinct = len(hosts)
    if n_distinct == 0:
        raise SystemExit("cfg3: no pinned host memory at all: " + str(refusal))

    def fill(job):
        l, e = job
        edg.pack_expert(desc0, synth.expert_tensors(cfg, l, e), hosts[l].numpy()[e])

    t_fill = time.time()
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
        list(ex.map(fill, [(l, e) for l in range(n_distinct) for e in range(E)]))
    t_fill = time.time() - t_fill
    hosts = [hosts[l % n_distinct] for l in range(L)]
    lor = [layer_io.lora_to_device(desc0, [synth.lora_tensors(cfg, l, 0)]) for l in range(L)]
    loras = [lo[0] for lo in lor]
    W = torch.from_numpy(np.stack([synth.prerouter_weights(cfg, l) for l in range(L)])).cuda()
    n_x = tokens + warm + 1
    X_iid = np.stack([synth.hidden_states(cfg, n_x, layer=l, stream=400) for l in range(L)])
    X_ar1 = np.stack([synth.hidden_states_ar1(cfg, n_x, 0.6, layer=l, stream=401) for l in range(L)])
    fit = _h2d_fit(R)
    arms = {}
    order = [("iid", "resident_S256", E, True), ("iid", "prefetch_S8", 8, True), ("iid", "on_demand_S8", 8, False),
             ("iid", "prefetch_S32", 32, True), ("ar1", "prefetch_S8", 8, True), ("ar1", "on_demand_S8", 8, False),
             ("ar1", "prefetch_S32", 32, True), ("ar1", "lru_S256", E, True),
             # the hot executor path (LRU-resident hot set, misses fetched by the SMs inside the step)
             ("ar1", "hot_S64", 64 + K, True), ("iid", "hot_S64", 64 + K, True), ("ar1", "hot_S64_k4", 64 + 4, True)]
    for routing, name, S, prefetch in order:
        Xn = X_iid if routing == "iid" else X_ar1
        X = layer_io.bits_to_device(Xn, torch.bfloat16)                     # [L][n_x][H]
        Xt = [X[:, t].contiguous() for t in range(n_x)]
        hot = name.startswith("hot")
        Kd = 4 if name.endswith("k4") else K                                # K = 4: the 35B tier's shipped profile
        d = edg.make_desc(cfg, n_slots=S, out_dtype="f32", K=Kd)
        slots = torch.empty((L, S, R), dtype=torch.uint8, device="cuda")
        tables = torch.empty((L, E), dtype=torch.int32, device="cuda")
        store = edg.Store(d, hosts, slots, tables, loras, torch.cuda.Stream())
        if hot:
            store.set_hot(True, 1)
        if name == "resident_S256":
            for l in range(L):
                for e0 in range(0, E, 64):
                    edg.stage_experts_to_slots(store, l, np.arange(e0, e0 + 64, dtype=np.int32))
            torch.cuda.synchronize()
        dec = StackDecoder(d, store, W, prefetch=prefetch)
        dec.prime(Xt[n_x - 1])
        Y = torch.zeros((L, H), dtype=torch.float32, device="cuda")
        for t in range(warm):
            dec.step(t, Xt[t], Y)
        torch.cuda.synchronize()
        store.time_waits(True)
        base = store.stats()
        prev_sets, overlap = None, []
        e0_, e1_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0_.record()
        for t in range(warm, warm + tokens):
            dec.step(t, Xt[t], Y)
        e1_.record()
        torch.cuda.synchronize()
        ms = e0_.elapsed_time(e1_) / tokens
        wait_ms, n_waits = store.exposed_wait_ms()
        st = store.stats()
        staged = (st["hits"] - base["hits"]) + (st["misses"] - base["misses"])
        arms[f"{routing}/{name}"] = {
            "ms_per_token": round(ms, 4), "tok_per_s": round(1e3 / ms, 1),
            "exposed_copy_ms_per_token": round(wait_ms / tokens, 4),
            "exposed_copy_how": "CUDA events around every wait of a compute stream on a layer's copy-done event",
            "waits_per_token": round(n_waits / tokens, 2),
            "copies_per_token": round((st["misses"] - base["misses"]) / tokens, 2),
            "hit_rate": round((st["hits"] - base["hits"]) / max(1, staged), 4),
            "MiB_copied_per_token": round((st["bytes_copied"] - base["bytes_copied"]) / tokens / 2 ** 20, 1),
            "hbm_GBps_on_expert_bytes": round(L * Kd * R / (ms * 1e-3) / 1e9, 1)}
        if hot:
            hs = store.hot_stats()
            arms[f"{routing}/{name}"].update({"K": Kd, "hot_slots": S - Kd, "admitted_per_token": round(hs["admitted"] / (tokens + warm), 2),
                                              "MiB_fetched_by_SMs_per_token": round(hs["bytes_direct"] / (tokens + warm) / 2 ** 20, 1)})
        assert edg.workspace_status(dec.ws) == 0 and bool(torch.isfinite(Y).all())
        store.close()
        del slots, tables, dec, X, Xt
        torch.cuda.empty_cache()
    head = arms["iid/prefetch_S8"]
    print(json.dumps({"metric": "expert_stack_decode_tok_per_s", "value": head["tok_per_s"], "unit": "tok/s",
                      "n_gpus": 1, "steps": tokens, "warmup": warm, "higher_is_better": True, "data": "synthetic",
                      "config": {"workload": "cfg3: 40-layer expert stack, batch-1 decode, pinned-host store -> HBM slot pool",
                                 "host_store_bytes": n_distinct * E * R, "distinct_host_layers": n_distinct,
                                 "pinned_refusal": refusal, "host_fill_s": round(t_fill, 1), "tokens": tokens,
                                 "routing": {"iid": "hidden states independent N(0,1) per token",
                                             "ar1": "x[t+1] = 0.6 x[t] + 0.8 eps: consecutive tokens share part of their routed set"},
                                 "host_loop": "edg_stack_decode_token (C): routing read from the kernels' pinned-host mirror, no stream synchronisation"},
                      "h2d_copy_fit": fit, "arms": arms}))


def run_prefill_stream(args):
    """Whole-layer prefill (Sec. 3.1, executor path 4): 4096 tokens through `depth` layers whose experts
    come from the pinned-host tier one whole layer per copy, into a double buffer of two pool layers;
    the load of layer l+1 overlaps the grouped FFN of layer l.  Arms: overlapped, and load-then-compute."""
    import torch
    from paper_2609_18063_b200 import build
    build.build()
    import paper_2609_18063_b200 as edg
    from paper_2609_18063_b200 import layer_io
    cfg = synth.CONFIGS["cfg5"]
    T, K, E, H, I = cfg.T, cfg.K, cfg.E, cfg.H, cfg.I
    depth = max(4, min(args.steps, 12))
    desc = edg.make_desc(cfg, n_slots=E, out_dtype="f32")
    R = edg.record_bytes(desc)
    hosts = build_instances(edg, layer_io, cfg, desc, depth, 0)
    lor = [layer_io.lora_to_device(desc, [synth.lora_tensors(cfg, l, 0)]) for l in range(depth)]
    pool = torch.empty((2, E, R), dtype=torch.uint8, device="cuda")
    tables = torch.empty((2, E), dtype=torch.int32, device="cuda")
    store = edg.Store(desc, hosts[:2], pool, tables, None, torch.cuda.Stream())
    x = layer_io.bits_to_device(synth.hidden_states(cfg, T, stream=300), torch.bfloat16)
    logits = torch.from_numpy(synth.zipf_router_logits(cfg, T)).cuda()
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    y = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(desc, T)
    st = torch.cuda.current_stream()

    def layer(l):
        p = l % 2
        store.wait_staged(p, st)
        edg.softmax_topk_rows(desc, logits, T, inds, gates)
        edg.moe_expert_ffn_int4_lora(desc, pool[p], tables[p], T, inds, None, gates, x, lor[l][0], y, ws)
        store.mark_computed(p, st)

    def run(overlap):
        store.load_whole_layer(0, hosts[0])
        torch.cuda.synchronize()
        store.time_waits(True)
        store.exposed_wait_ms()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for l in range(depth):
            if overlap and l + 1 < depth:
                store.load_whole_layer((l + 1) % 2, hosts[l + 1])
            layer(l)
            if not overlap and l + 1 < depth:                 # serial: the load starts when the layer has finished
                torch.cuda.synchronize()
                store.load_whole_layer((l + 1) % 2, hosts[l + 1])
        e1.record()
        torch.cuda.synchronize()
        wait_ms, n = store.exposed_wait_ms()
        return e0.elapsed_time(e1) / depth, wait_ms / depth

    run(True)
    arms = {}
    for name, ov in (("overlapped", True), ("load_then_compute", False), ("overlapped_again", True)):
        ms, wait = run(ov)
        arms[name] = {"ms_per_layer": round(ms, 3), "exposed_load_ms_per_layer": round(wait, 3),
                      "tok_per_s": round(T / (ms * 1e-3), 1), "host_link_GBps": round(E * R / (ms * 1e-3) / 1e9, 1)}
    assert edg.workspace_status(ws) == 0 and bool(torch.isfinite(y).all())
    print(json.dumps({"metric": "moe_layer_prefill_streamed_tok_per_s", "value": arms["overlapped"]["tok_per_s"], "unit": "tok/s",
                      "n_gpus": 1, "steps": depth, "warmup": depth, "higher_is_better": True, "data": "synthetic",
                      "config": {"workload": "whole-layer prefill: 4096 tokens (cfg5 routing), one 453 MB copy per layer from pinned host memory into a two-layer pool",
                                 "depth": depth, "bytes_per_layer": E * R}, "arms": arms}))


def run_sigmoid_group(args):
    """The paper's second routing family (Appendix A, sigmoid-group; 8B tier: E = 128, n = 8 groups,
    keep 4, K = 8, scale 2.5) on given logits: rows per second and bytes per second of the one kernel."""
    import torch
    import paper_2609_18063_b200 as edg
    peak, how = _peaks()
    E, K, n, G, T = 128, 8, 8, 4, 1 << 19           # 268 MB of logits: larger than L2
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    logits = torch.randn((T, E), generator=g, device="cuda", dtype=torch.float32) * 2.0
    bias = (torch.rand((E,), generator=g, device="cuda", dtype=torch.float32) - 0.5) * 0.1
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    steps, warmup = max(1, min(args.steps, 50)), max(args.warmup, 3)
    for _ in range(warmup):
        edg.sigmoid_group_topk_rows(logits, T, E, K, n, G, 2.5, bias, inds, gates)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        edg.sigmoid_group_topk_rows(logits, T, E, K, n, G, 2.5, bias, inds, gates)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert int(inds.min()) >= 0 and int(inds.max()) < E and abs(float(gates[0].sum()) - 2.5) < 1e-4
    alg = T * (E * 4 + K * 8)
    achieved = alg / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "sigmoid_group_routing_rows_per_s", "value": round(T / (ms * 1e-3), 1), "unit": "rows/s",
                      "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": round(ms, 5), "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": "sigmoid-group routing, 8B-tier shape: E=128, 8 groups keep 4, top-8, scale 2.5, 524288 rows of logits",
                                 "l2": "268 MB of logits per launch exceed the 126 MB L2"},
                      "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                                   "frac": round(achieved / peak, 4), "traffic": None, "peak_kind": how,
                                   "algorithmic_bytes_per_launch": alg},
                      "gpu_launches": steps}))


def run_mlp_head(args):
    """The full prerouter head (Sec. 3.2: fc1 -> erf-gelu -> fc2 + linear residual path; feature = hidden
    state and two K-hot vectors) for many (head, state) pairs in one launch, as in the paper's single
    flush: 64 heads of the 35B-tier shape (H + 2E = 2560, width 512, fp16), 252 MB of head weights."""
    import torch
    import paper_2609_18063_b200 as edg
    from workloads import synth
    from paper_2609_18063_b200 import layer_io
    peak, how = _peaks()
    cfg = synth.CONFIGS["cfg2"]
    desc = edg.make_desc(cfg, n_slots=cfg.E)
    E, K, H, D, NH = cfg.E, cfg.K, cfg.H, 512, 64
    hw = [synth.mlp_head_weights(cfg, l % 4, D) for l in range(4)]         # four distinct heads, tiled to 64
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    tile = lambda k: dev(np.stack([hw[l % 4][k] for l in range(NH)]))
    W1, b1, W2, b2 = tile("W1"), tile("b1"), tile("W2"), tile("b2")
    Wr = dev(np.stack([synth.prerouter_weights(cfg, l % 4) for l in range(NH)]))
    X = layer_io.bits_to_device(synth.hidden_states(cfg, NH, stream=600), torch.bfloat16)
    rng = np.random.default_rng(9)
    cur = dev(np.stack([np.sort(rng.choice(E, K, replace=False)) for _ in range(NH)]).astype(np.int32))
    prev = dev(np.stack([np.sort(rng.choice(E, K, replace=False)) for _ in range(NH)]).astype(np.int32))
    inds = torch.zeros((NH, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((NH, K), dtype=torch.float32, device="cuda")
    steps, warmup = max(1, min(args.steps, 200)), max(args.warmup, 3)
    call = lambda: edg.prerouter_mlp_topk(desc, W1, b1, W2, b2, Wr, D, X, cur, prev, NH, inds, gates, None)
    for _ in range(warmup):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert abs(float(gates.sum()) - NH) < 1e-2
    alg = NH * (D * (H + 2 * E) * 2 + E * D * 2 + E * H * 2 + (D + E) * 2 + H * 2)
    achieved = alg / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "prerouter_mlp_heads_per_s", "value": round(NH / (ms * 1e-3), 1), "unit": "heads/s",
                      "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": round(ms, 5), "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "fp16 weights, fp32 accumulate", "data": "synthetic",
                      "config": {"workload": "full prerouter head, 35B-tier shape (feature 2560, width 512, E=256, top-8), 64 heads per launch",
                                 "l2": "252 MB of head weights per launch exceed the 126 MB L2"},
                      "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                                   "frac": round(achieved / peak, 4), "traffic": None, "peak_kind": how,
                                   "algorithmic_bytes_per_launch": alg},
                      "gpu_launches": steps}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10240)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--impl", choices=["b200", "reference"], default="b200")
    ap.add_argument("--instances", type=int, default=8, help="independently seeded resident layer instances")
    ap.add_argument("--e2e-steps", type=int, default=400)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dependent", action="store_true")
    ap.add_argument("--no-secondary", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", choices=["cfg2", "cfg3", "cfg4", "cfg5", "sigmoid_group", "mlp_head", "prefill_stream"], default="cfg2",
                    help="cfg2 is the headline line; the others print their own line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "cfg3":
        run_cfg3(args)
    elif args.workload == "cfg4":
        run_cfg4(args)
    elif args.workload == "cfg5":
        run_cfg5(args)
    elif args.workload == "sigmoid_group":
        run_sigmoid_group(args)
    elif args.workload == "mlp_head":
        run_mlp_head(args)
    elif args.workload == "prefill_stream":
        run_prefill_stream(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
