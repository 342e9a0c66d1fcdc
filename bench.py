#!/usr/bin/env python
"""Benchmark of the fused routed-MoE decode step on B200.

One "step" = one layer-step of the whole operator (router, top-k, input quantisation, gate/up projection,
SwiGLU + requantisation, down projection, weighted reduction) = one launch of the persistent kernel.
Default workload: the Qwen3-30B-A3B-like layer (H=2048, E=128, top-8, I=768) at T=1.  Consecutive steps rotate
over L distinct layer copies (different weights and routers) so that every step streams its experts from HBM,
not from L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--tokens T] [--regime R] [--impl reference]

Prints ONE JSON line.  `value` is microseconds per layer-step with all inputs resident in HBM; `e2e` is the same
through the public API with the step's input copied from pinned host memory and the result copied back.
`--impl reference` times the CPU oracle (the reference arm) on the same workload.
With N > 1 (torchrun) every rank runs an independent replica: the operator does not shard (no collectives).
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

METRIC = "us_per_moe_layer_step"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the step's kernel from the ncu
# captures summarised under profiles/; keyed by (config, tokens).  None where no capture exists.
NCU_TRAFFIC_BYTES = {
    ("c1_tiny", 1): 3.507e6,                         # profiles/moe_fused_kernel_c1_tiny_t1.md
    ("c2_qwen3_30b_a3b", 1): 39.221e6 + 0.097e6,     # profiles/moe_fused_kernel_c2_qwen3_t1.md
    ("c2_qwen3_30b_a3b", 2): 76.986e6 + 2.952e6,     # profiles/moe_fused_kernel_c2_qwen3_t2.md
    ("c2_qwen3_30b_a3b", 4): 149.72e6 + 4.71e6,      # profiles/moe_fused_kernel_c2_qwen3_t4.md
    ("c2_qwen3_30b_a3b", 8): 251.81e6 + 6.10e6,      # profiles/moe_fused_kernel_c2_qwen3_t8.md
    ("c2_qwen3_30b_a3b", 16): 379.39e6 + 4.64e6,     # profiles/moe_decode_kernel_c2_qwen3_t16.md
    ("c2_qwen3_30b_a3b", 64): 601.9e6 + 5.6e6,       # profiles/moe_decode_kernel_c2_qwen3_t64.md
    ("c4_mixtral_8x7b", 1): 365.72e6 + 5.35e6,       # profiles/moe_fused_kernel_c4_mixtral_t1.md
    ("c4_mixtral_8x7b", 64): 1416.3e6 + 6.8e6,       # profiles/moe_decode_kernel_c4_mixtral_t64.md
    ("c5_deepseek_v3[E=16]", 1): 356.76e6 + 4.67e6,  # profiles/moe_decode_kernel_c5like_e16_t1.md
    ("c5_deepseek_v3[E=32]", 1): 353.59e6 + 5.62e6,  # profiles/moe_fused_kernel_c5like_e32_t1.md
    ("c5_deepseek_v3[E=64]", 8): 1680.1e6 + 4.8e6,   # profiles/moe_decode_kernel_c5like_e64_t8.md
}


# (config, tokens, regime) cells measured after the headline in the default run
CELLS = [("c1_tiny", 1, "natural"), ("c2_qwen3_30b_a3b", 2, "natural"), ("c2_qwen3_30b_a3b", 4, "natural"),
         ("c2_qwen3_30b_a3b", 8, "natural"), ("c2_qwen3_30b_a3b", 8, "same"), ("c4_mixtral_8x7b", 1, "natural"),
         ("c5_deepseek_v3", 1, "natural"), ("c5_deepseek_v3", 8, "natural")]


def kernel_name(info, T, shape=None):
    """Name of the kernel instantiation a plan launches for T tokens."""
    if info.get("fused"):
        tc = 1 if T <= 1 else 2 if T <= 2 else 4 if T <= 4 else 8 if T <= 8 else 16
        if shape is None:
            return f"moe_fused_kernel<{tc}>"
        # the instantiation with the unit-sharing code runs where a step can have more units than clusters
        clusters = info["grid"] if info.get("pairs_at_runtime") else info["grid"] // max(1, info["cluster"])
        split = min(shape.E, T * shape.top_k) * (shape.I // 128) > clusters and (shape.H // 128) % max(1, info["cluster"]) == 0
        return f"moe_fused_kernel<{tc}, {1 if split else 0}>"
    return f"moe_decode_kernel<N={info['n_hw']}>"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--config", default="c2_qwen3_30b_a3b")
    ap.add_argument("--schedule", default="", help="schedule table written by paper_2609_04244_b200.tune (JSON)")
    ap.add_argument("--tokens", type=int, default=1)
    ap.add_argument("--regime", default="natural", choices=["natural", "same", "disjoint"])
    ap.add_argument("--layers", type=int, default=0, help="distinct layer copies to rotate over (0 = auto)")
    ap.add_argument("--experts", type=int, default=0,
                    help="override the number of experts E (same per-expert shapes): a small case for profiler captures")
    ap.add_argument("--no-graph", action="store_true", help="launch the timed steps directly instead of from CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cells", action="store_true", help="skip the extra (config, tokens) cells measured after the headline")
    return ap.parse_args()


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples = []
        self.stop = threading.Event()
        self.thread = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None

    def _run(self):
        nv = self.nv
        while not self.stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self.ok:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()

    def finish(self, t0=None, t1=None):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        self.stop.set()
        self.thread.join(timeout=1.0)
        nv = self.nv
        inside = [s for s in self.samples if t0 is None or (t0 <= s[0] <= t1)]
        use = inside if inside else self.samples[-5:]
        mhz = sorted(s[1] for s in use)
        bits = 0
        for s in use:
            bits |= s[2]
        names = []
        table = [("hw_slowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("sw_thermal_slowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("sw_power_cap", "nvmlClocksThrottleReasonSwPowerCap")]
        for name, attr in table:
            if bits & getattr(nv, attr, 0):
                names.append(name)
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": self.max_mhz, "reasons": names,
                "samples": len(use), "window": "timed region" if inside else "around timed region"}


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity when not running under torchrun)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(us_per_step_per_rank: float, world: int) -> float:
    """Replicas run side by side: N ranks finish N layer-steps in the time one rank needs for one."""
    return us_per_step_per_rank / world


def oracle_inputs(d, ids):
    """Host copies of exactly what the oracle needs: hidden, router, bias and the selected experts' weights."""
    import numpy as np
    import torch
    used = np.unique(ids)
    emap = np.full(d["Wr"].shape[0], -1, np.int32)
    emap[used] = np.arange(len(used))
    sel = torch.as_tensor(used, device=d["W13q"].device, dtype=torch.long)
    u16 = lambda t: t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    return dict(hidden=u16(d["hidden"]), Wr=u16(d["Wr"]), bias=None if d["bias"] is None else d["bias"].cpu().numpy(),
                W13q=d["W13q"][sel].cpu().numpy(), W13s=d["W13s"][sel].cpu().numpy(), W2q=d["W2q"][sel].cpu().numpy(),
                W2s=d["W2s"][sel].cpu().numpy(), emap=emap)


def time_oracle(shape, host, reps_budget_s=12.0, max_reps=50):
    """Wall-clock of the CPU oracle, as it stands, on one layer-step; returns (us per step, reps, threads)."""
    import oracle
    reps, total = 0, 0.0
    while reps < max_reps and (reps < 2 or total < reps_budget_s):
        t0 = time.perf_counter()
        oracle.moe_forward(host["hidden"], host["Wr"], host["bias"], host["W13q"], host["W13s"], host["W2q"],
                           host["W2s"], top_k=shape.top_k, scoring=shape.scoring, renorm=shape.renorm,
                           expert_map=host["emap"])
        total += time.perf_counter() - t0
        reps += 1
    return total / reps * 1e6, reps, oracle.threads()


def run_reference(args, shape):
    """The reference arm: the CPU oracle on the bench workload (host cores), same metric and config keys."""
    import numpy as np
    import torch
    from paper_2609_04244_b200 import workloads as wl
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    T = args.tokens
    # inputs generated on the host: route first, then generate only the experts the oracle will touch
    seed = wl.workload_seed(shape, T, args.regime, 0)
    hidden = wl.make_hidden(shape, T, seed, "cpu")
    Wr, bias = wl.make_router(shape, seed, "cpu")
    Wr = wl.force_routing(Wr, hidden, shape.top_k, args.regime)
    u16 = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    rt = oracle.route_and_quantize(u16(hidden), u16(Wr), None if bias is None else bias.numpy(), shape.top_k,
                                   shape.scoring, shape.renorm)
    used = np.unique(rt["ids"])
    w = wl.make_expert_weights(shape, seed, "cpu", experts=[int(e) for e in used])
    d = {"hidden": hidden, "Wr": Wr, "bias": bias, **w}
    host = oracle_inputs(d, rt["ids"])
    steps, warm = max(1, min(args.steps, 20)), max(0, min(args.warmup, 2))
    for _ in range(warm):
        time_oracle(shape, host, reps_budget_s=0.0, max_reps=2)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.moe_forward(host["hidden"], host["Wr"], host["bias"], host["W13q"], host["W13s"], host["W2q"],
                           host["W2s"], top_k=shape.top_k, scoring=shape.scoring, renorm=shape.renorm,
                           expert_map=host["emap"])
    us = (time.perf_counter() - t0) / steps * 1e6
    sample = f"{steps} full layer-steps at T={T} (steps capped at 20 for the CPU arm)"
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{shape.name} T={T} regime={args.regime}", "H": shape.H, "E": shape.E, "I": shape.I,
                       "top_k": shape.top_k, "tokens": T},
            "cpu_baseline": {"value": us, "unit": "us", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    from paper_2609_04244_b200 import workloads as wl
    shape = wl.SHAPES[args.config]
    if args.experts:
        import dataclasses
        shape = dataclasses.replace(shape, E=args.experts, name=f"{shape.name}[E={args.experts}]")
    if args.impl == "reference":
        run_reference(args, shape)
        return

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2609_04244_b200 import MoEPlan

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fused kernel has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    T, K, W = args.tokens, args.steps, max(args.warmup, 3)
    schedule = None
    if args.schedule:
        import json as _json
        with open(args.schedule) as f:
            schedule = _json.load(f)

    def measure(shape, T, regime, K, W, keep=False):
        """Device-resident timing of K layer-steps of `shape` at T tokens: CUDA-graph replay over distinct layer copies."""
        # enough distinct layer copies that the bytes streamed between two uses of a copy exceed 2x L2 (126 MB)
        per_step = wl.algorithmic_bytes(shape, T, min(shape.E, int(round(wl.expected_unique_experts(shape.E, shape.top_k, T)))))
        free_b, _ = torch.cuda.mem_get_info()
        layer_bytes = shape.E * shape.bytes_per_expert
        L = args.layers or max(2, min(16, -(-2 * 126 * 2**20 // per_step) + 1))
        L = max(1, min(L, int(0.6 * free_b // layer_bytes)))
        layers = [wl.make_layer(shape, T, regime=regime, layer=rank * 64 + l, device=dev) for l in range(L)]
        plan = MoEPlan(shape.H, shape.E, shape.I, shape.top_k, shape.scoring, shape.renorm, T_max=T, schedule=schedule)
        info = plan.info(T)
        outs = [torch.empty((T, shape.H), dtype=torch.bfloat16, device=dev) for _ in range(L)]

        def step(i):
            d = layers[i % L]
            plan.forward(d["hidden"], d["Wr"], d["bias"], d["W13q"], d["W13s"], d["W2q"], d["W2s"], out=outs[i % L])

        # unique experts per layer copy (from the kernel's own routing) -> algorithmic bytes per step
        uniq = []
        tpl = plan.tokens_per_launch()
        ids_last = None
        for l in range(L):
            d = layers[l]
            ids_all = []
            for lo in range(0, T, tpl):              # the debug entry point takes one launch's worth of tokens
                dbg = plan.forward_debug(d["hidden"][lo:lo + tpl].contiguous(), d["Wr"], d["bias"], d["W13q"], d["W13s"],
                                         d["W2q"], d["W2s"])
                plan.sync_status()
                ids_all.append(dbg["ids"])
            ids_last = torch.cat(ids_all)
            uniq.append(int(torch.unique(ids_last).numel()))
        bytes_per_step = float(np.mean([wl.algorithmic_bytes(shape, T, u) for u in uniq]))
        launches_per_step = -(-T // tpl)

        # The timed steps are replayed from CUDA graphs (Section 4.1 of the paper times graph replays): a graph holds
        # up to 1000 consecutive steps, so the host's per-call cost (Python, ctypes, launch) is not what is measured.
        for i in range(W):
            step(i)
        torch.cuda.synchronize()

        def capture(first, n):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(n):
                    step(first + i)
            return g

        class _Direct:                                      # --no-graph: same interface, plain launches
            def __init__(self, first, n):
                self.first, self.n = first, n

            def replay(self):
                for i in range(self.n):
                    step(self.first + i)

        if args.no_graph:
            capture = _Direct
        CH = 1000
        graphs, done = [], 0
        full = capture(W, CH) if K >= CH else None          # replayed K // CH times; the layer rotation inside it is
        while done + CH <= K:                               # what keeps L2 cold, not the seam between two replays
            graphs.append(full)
            done += CH
        if K - done:
            graphs.append(capture(W + done, K - done))
        for g in {id(g): g for g in graphs}.values():       # one untimed replay of each graph (first-launch upload)
            g.replay()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        sampler = ClockSampler(local)
        sampler.start()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t_wall0 = time.perf_counter()
        torch.cuda.nvtx.range_push("timed_region")      # lets a profiler restrict itself to the timed steps
        ev0.record(stream)
        for g in graphs:
            g.replay()
        ev1.record(stream)
        torch.cuda.synchronize()
        torch.cuda.nvtx.range_pop()
        t_wall1 = time.perf_counter()
        if world > 1:
            dist.barrier()
        ms = ev0.elapsed_time(ev1)
        if t_wall1 - t_wall0 < 0.25:        # timed region too short for a clock sample: keep the same load running briefly
            t_end = time.perf_counter() + 0.3
            while time.perf_counter() < t_end:
                graphs[0].replay()
                torch.cuda.synchronize()
            clocks = sampler.finish()
            clocks["window"] = "timed region + 0.3 s of the same load"
        else:
            clocks = sampler.finish(t_wall0, t_wall1)
        plan.sync_status()
        res = {"ms": ms, "K": K, "L": L, "info": info, "uniq": uniq, "bytes_per_step": bytes_per_step,
               "launches_per_step": launches_per_step, "clocks": clocks}
        if keep:
            res.update(plan=plan, layers=layers, ids_last=ids_last)
        else:
            plan.close()
            del layers, outs, graphs, full
            torch.cuda.empty_cache()
        return res

    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    head = measure(shape, T, args.regime, K, W, keep=True)
    plan, layers, ids_last, L = head["plan"], head["layers"], head["ids_last"], head["L"]
    info, uniq, bytes_per_step, launches_per_step, clocks, ms = (head[k] for k in ("info", "uniq", "bytes_per_step", "launches_per_step", "clocks", "ms"))

    # end to end: the step's input comes from pinned host memory, the result goes back to the host
    e2e = None
    if not args.no_e2e:
        # through the public C-ABI call that takes HOST activations (moe_forward_host): per step one pinned
        # host-to-device copy of the hidden state, the kernel, one device-to-host copy of the output, and a stream
        # synchronisation because the caller consumes the result before the next step
        h_in = [layers[l]["hidden"].cpu().pin_memory() for l in range(L)]
        h_out = torch.empty((T, shape.H), dtype=torch.bfloat16).pin_memory()

        bound = [plan.bind_forward_host(h_in[l], layers[l]["Wr"], layers[l]["bias"], layers[l]["W13q"], layers[l]["W13s"],
                                        layers[l]["W2q"], layers[l]["W2s"], h_out, stream) for l in range(L)]
        sync = stream.synchronize

        def e2e_step(i):
            bound[i % L]()          # moe_forward_host: H2D copy of the step's input, the kernel (writes h_out itself)
            sync()                  # the caller consumes the result before the next step

        Ke = min(K, 2000)
        for i in range(W):
            e2e_step(i)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(Ke):
            e2e_step(W + i)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1)
        e2e = {"ms": e2e_ms, "steps": Ke}
        plan.sync_status()

    # More cells of the (config, tokens) table, measured in this same run with the same protocol (graph replay, layer
    # rotation, clocks sampled per cell): the headline stays the line's `value`.
    cells = None
    if world == 1 and not args.no_cells and args.config == "c2_qwen3_30b_a3b" and T == 1 and args.regime == "natural" and not args.experts:
        peak_c, _ = peak_hbm()
        cells = []
        Kc = max(200, min(K, 1000))
        for name, Tc, regime in CELLS:
            shp = wl.SHAPES[name]
            r = measure(shp, Tc, regime, Kc, W)
            us = r["ms"] * 1e3 / Kc
            gbs = r["bytes_per_step"] / (us * 1e-6) / 1e9
            cells.append({"workload": f"{name} T={Tc} regime={regime}", "us": us, "steps": Kc,
                          "algorithmic_bytes_per_step": r["bytes_per_step"], "achieved_gbs": gbs, "frac": gbs / peak_c,
                          "traffic": NCU_TRAFFIC_BYTES.get((name, Tc)) if regime == "natural" else None,
                          "unique_experts_mean": float(np.mean(r["uniq"])), "layer_copies": r["L"],
                          "variant": kernel_name(r["info"], Tc, shp), "cluster": r["info"]["cluster"], "stages": r["info"]["stages"],
                          "clocks": {k: r["clocks"].get(k) for k in ("sm_mhz", "sm_max_mhz", "reasons")}})

    ms, e2e_ms_max = max_over_ranks([ms, e2e["ms"] if e2e else 0.0], dev)
    if e2e:
        e2e["ms"] = e2e_ms_max

    if rank == 0:
        us_step = ms * 1e3 / K                     # per rank; replicas run side by side
        value = whole_job_value(us_step, world)    # whole-job: microseconds per layer-step over all replicas
        kernel_us = us_step / launches_per_step
        peak, peak_kind = peak_hbm()
        achieved = bytes_per_step / launches_per_step / (kernel_us * 1e-6) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": "us", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": us_step / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp8_e4m3 x fp8_e4m3 -> f32", "data": "synthetic",
            "config": {"workload": f"{shape.name} T={T} regime={args.regime}", "H": shape.H, "E": shape.E, "I": shape.I,
                       "top_k": shape.top_k, "tokens": T, "unique_experts_mean": float(np.mean(uniq)),
                       "layer_copies": L, "l2": f"rotates over {L} distinct layer copies "
                       f"({L * bytes_per_step / 2**20:.0f} MiB streamed between reuses, L2 is 126 MiB)",
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "grid": info["grid"], "stages": info["stages"], "n_hw": info["n_hw"],
                       "variant": kernel_name(info, T, shape), "cluster": info["cluster"],
                       "launch": "direct launches" if args.no_graph else "CUDA graph replay, one kernel node per step"},
            "achieved_gbs": achieved, "algorithmic_bytes_per_step": bytes_per_step,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"of {peak_kind}", "kernel": kernel_name(info, T, shape), "kernel_us": kernel_us,
                         "traffic": NCU_TRAFFIC_BYTES.get((shape.name, T))},
            "gpu_launches": K * launches_per_step,
            "clocks": clocks,
        }
        if e2e:
            eus = whole_job_value(e2e["ms"] * 1e3 / e2e["steps"], world)
            line["e2e"] = {"value": eus, "unit": "us", "h2d_bytes_per_step": 2 * T * shape.H,
                           "d2h_bytes_per_step": 2 * T * shape.H, "steps": e2e["steps"]}
        if world == 1 and not args.no_cpu_baseline:
            d = layers[L - 1]
            host = oracle_inputs(d, ids_last.cpu().numpy())
            us_cpu, reps, thr = time_oracle(shape, host)
            line["cpu_baseline"] = {"value": us_cpu, "unit": "us", "cores": thr, "kind": "oracle",
                                    "sample": f"{reps} full layer-steps of the same workload (T={T}), mean"}
        if cells is not None:
            line["cells"] = cells
        print(json.dumps(line), flush=True)
    plan.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
