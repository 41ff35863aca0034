#!/usr/bin/env python
"""Decode-throughput benchmark of the MoE layer step on one B200 (or N replicas).

A step is one decode token through every layer of the stack (router + top-K, predictor,
cache/prefetch where the stack is offloaded, routed SwiGLU FFN, residual) for one batch of
synthetic input.  Default workload: the Mixtral-8x7B-shaped bf16 stack with all experts
resident (about 90 GB of weights), batch 1.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C1] [--batch B]
  python bench.py --impl reference ...     # the CPU oracle on the host cores

Prints one JSON line.  `value` is device-timed with inputs resident in HBM; `e2e` is the
same metric through the public API with pinned host buffers copied in and out every step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from datagen import stacks  # noqa: E402

METRIC, UNIT = "decode_tokens_per_s", "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period=0.05):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.reasons |= {n for bit, n in names.items() if r & bit}
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def load_stack(cfg, batch, dev, **kw):
    import paper_2606_15453_b200 as P
    st = P.Stack.from_config(cfg, max_batch=batch, **kw)
    for l, w in enumerate(stacks.router_weights(cfg)):
        st.load_router(l, w)
    for l in range(cfg.n_layers):
        for shared, n in ((False, cfg.n_experts), (True, cfg.n_shared)):
            for e in range(n):
                w = stacks.expert_weights(cfg, l, e, shared, device=dev)
                sc = torch.cat([w["gate_scale"], w["up_scale"], w["down_scale"]]) \
                    if cfg.dtype == "fp8" else None
                # load_experts copies at once, outside torch's streams: the generator must be done
                torch.cuda.current_stream().synchronize()
                st.load_experts(l, e, w["gate"], w["up"], w["down"], sc, shared)
        del w
    return st


def algorithmic_bytes(cfg, ids_per_layer):
    """Bytes the step must stream: distinct routed experts (+ shared) and the router, per layer."""
    total = 0
    for ids in ids_per_layer:
        total += (len(np.unique(ids)) + cfg.n_shared) * cfg.expert_bytes + cfg.router_bytes
    return total


def cpu_oracle_sample(cfg, batch, layers, tokens, dev):
    """Time the CPU oracle (as it stands) on the first `tokens` decode steps through the first
    `layers` layers; expert weights are regenerated from the seed (same bits as the GPU's)."""
    import oracle as O
    from oracle.stack import OracleStack
    store = {}

    def experts(l, e, shared=False):
        if (l, e, shared) not in store:
            w = stacks.expert_weights(cfg, l, e, shared, device=dev)
            store[(l, e, shared)] = {k: v.cpu().contiguous() for k, v in w.items()}
        return store[(l, e, shared)]

    orc = OracleStack(cfg, stacks.router_weights(cfg), experts, batch=batch, cache_slots=0)
    x = stacks.token_inputs(cfg, batch, tokens).numpy()
    spent = []
    for t in range(tokens):
        h, dt = x[t], 0.0
        for l in range(layers):
            # fetch the weights this step needs outside the timed part
            routes = orc.route(l, h)
            for r in routes:
                for e in r["ids"]:
                    experts(l, int(e))
            for s in range(cfg.n_shared):
                experts(l, s, True)
            t0 = time.perf_counter()
            res = orc.layer_step(l, h)
            dt += time.perf_counter() - t0
            h = res["h_out"]
        spent.append(dt)
    return spent, O.get_threads()


def workload_config(cfg, batch, world):
    """The workload both arms (this library, the CPU oracle) are timed on: identical keys and values."""
    return {"workload": cfg.name, "batch": batch, "layers": cfg.n_layers, "experts": cfg.n_experts,
            "top_k": cfg.top_k, "hidden": cfg.hidden, "inter": cfg.inter, "profile_tokens": cfg.profile_tokens,
            "parallelism": f"replicas x{world}", "l2": "inputs_larger_than_l2"}


def run_reference(args, cfg, batch):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    layers = min(cfg.n_layers, args.ref_layers)
    spent, cores = cpu_oracle_sample(cfg, batch, layers, args.warmup + args.steps, dev)
    timed = spent[args.warmup:]
    per_token = sum(timed) / len(timed) * cfg.n_layers / layers
    value = batch / per_token
    sample = (f"{args.steps} decode steps x first {layers} of {cfg.n_layers} layers, batch {batch}, "
              f"scaled to the full depth")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_token * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype,
        "data": "synthetic",
        "config": workload_config(cfg, batch, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def profile_value(name):
    """A figure recorded in an ncu summary under profiles/ ("<name>: <number>" on a line of its
    own), or None: the DRAM traffic in the roofline object comes from there, not from a literal here."""
    import glob
    import re
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        m = re.search(r"^" + re.escape(name) + r":\s*([0-9.eE+]+)\s*$", open(path).read(), flags=re.M)
        if m:
            return float(m.group(1)), os.path.basename(path)
    return None, None


def top_kernel_name(cfg, batch, args):
    """The kernel that dominates a decode step of this workload (one launch per step for resident stacks)."""
    dense = not args.no_dense and cfg.dtype in ("bf16", "fp8") and batch >= (args.dense_min_batch or 2)
    if cfg.cache_slots:   # per-layer kernels; the tensor-core ones read the slot store (no shared experts there)
        return "dense_group_kernel (gate/up)" if dense and cfg.n_shared == 0 else "gate_up_kernel"
    if dense:
        return "dense_group_kernel (gate/up)" if args.no_persistent else "decode_token_dense_kernel"
    epl = {"f32": 4, "bf16": 8, "fp8": 16}[cfg.dtype]
    fused = batch == 1 and not args.no_fused and cfg.hidden % epl == 0 and cfg.hidden <= 4096 and \
        cfg.hidden // epl in (64, 128, 256, 512)
    return "decode_token_fused_kernel" if fused else "decode_token_kernel"


def measure(cfg, batch, st, args, dev, world, stream, with_e2e):
    """Profiling steps, warm-up, K timed decode steps on resident inputs, an untimed pass that records
    the routing (for the algorithmic bytes), optionally the end-to-end pass.  Returns a dict."""
    import torch.distributed as dist
    L, K, H = cfg.n_layers, cfg.top_k, cfg.hidden
    steps, warmup = args.steps, args.warmup
    n_tok = cfg.profile_tokens + warmup + steps
    x_host = stacks.token_inputs(cfg, batch, n_tok).pin_memory()
    x_dev = x_host.to(dev)
    h_out = torch.empty(batch, H, device=dev)
    ids = torch.empty(L, batch, K, dtype=torch.int32, device=dev)
    pred = torch.empty(L, batch, st.max_pred, dtype=torch.int32, device=dev)
    npred = torch.empty(L, batch, dtype=torch.int32, device=dev)
    h_in = torch.empty(batch, H, device=dev)
    local = dev.index or 0

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    gap_cycles = int(args.inter_layer_gap_us * 1965)      # torch.cuda._sleep spins on the SM clock

    def decode(h_src):
        h_in.copy_(h_src)
        if gap_cycles <= 0:
            st.decode_token(h_in, h_out, ids, None, pred, npred)
            return
        for l in range(L):                                # per-layer entry point + attention stand-in
            st.decode_step(l, h_in if l == 0 else h_out, h_out, ids[l], None, pred[l], npred[l])
            torch.cuda._sleep(gap_cycles)

    t = 0
    for _ in range(cfg.profile_tokens + warmup):          # the profiling phase of Algorithm 1, then warm-up
        decode(x_dev[t])
        t += 1
    s0 = st.stats()
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for i in range(steps):
        decode(x_dev[t + i])
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    s1 = st.stats()

    # the routing of the same steps (it depends on the inputs only), for the algorithmic bytes
    ids_seen = []
    for i in range(steps):
        decode(x_dev[t + i])
        ids_seen.append(ids.cpu().numpy().copy())
    e2e_ms = None
    if with_e2e:
        out_host = torch.empty(batch, H).pin_memory()
        ids_host = torch.empty(L, batch, K, dtype=torch.int32).pin_memory()
        barrier()
        w0 = time.perf_counter()
        for i in range(steps):      # one library call per step: pinned input in, output and routing back
            st.decode_token_host(x_host[t + i], out_host, ids_host)
        e2e_ms = (time.perf_counter() - w0) * 1e3
        barrier()
    ms, e2e_ms = max_over_ranks([ms, e2e_ms or 0.0], world, dev)
    step_bytes = [algorithmic_bytes(cfg, a) for a in ids_seen]
    return dict(ms=ms, e2e_ms=e2e_ms, clocks=clocks, s0=s0, s1=s1, step_bytes=step_bytes, steps=steps,
                overlap=routing_overlap(ids_seen))


def max_over_ranks(values, world, device):
    """The slowest rank's figures: replicas run the same steps side by side, the job's time per step is
    the maximum over ranks (value = the tokens of all ranks over that time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def routing_overlap(ids_seen):
    """Mean number of experts two routings share: the same layer at consecutive decode steps of a
    sequence (temporal) and adjacent layers of one step (spatial); ids_seen: [T] arrays [L][B][K].
    Independent uniform routings would share K*K/N (the paper's random baseline, Section 3.2)."""
    a = np.stack(ids_seen)                                    # [T][L][B][K]
    def shared(u, v):                                         # [...][K] x [...][K] -> mean |u & v|
        return float((u[..., :, None] == v[..., None, :]).sum(axis=(-1, -2)).mean()) if u.size and v.size else None
    return {"temporal": shared(a[1:], a[:-1]), "spatial": shared(a[:, 1:], a[:, :-1])}


def summarise(cfg, batch, m, args, world, peak):
    """The fields shared by the headline line and the secondary records."""
    tokens = m["steps"] * batch * world
    value = tokens / (m["ms"] * 1e-3)
    step_gbs = statistics.mean(m["step_bytes"]) / (m["ms"] / m["steps"] * 1e-3) / 1e9
    s0, s1 = m["s0"], m["s1"]
    run = {k: s1[k] - s0[k] for k in ("runtime_steps", "routed", "predicted", "hits", "near_ties", "cache_hits",
                                      "cache_misses", "kernel_launches", "prefetch_issued", "prefetch_useful",
                                      "prefetch_wasted", "transfer_ms", "exposed_ms")}
    out = {"workload": cfg.name, "batch": batch, "value": value, "unit": UNIT, "ms_per_step": m["ms"] / m["steps"],
           "algorithmic_bytes_per_step": statistics.mean(m["step_bytes"]), "achieved_gbs": step_gbs,
           "frac": step_gbs / peak, "frac_of_8000": step_gbs / 8000.0, "kernel": top_kernel_name(cfg, batch, args),
           "clocks": m["clocks"], "gpu_launches": run["kernel_launches"],
           "predictor": {"recall": run["hits"] / max(run["routed"], 1), "precision": run["hits"] / max(run["predicted"], 1),
                         "mean_predicted": run["predicted"] / max(run["runtime_steps"], 1), "near_ties": run["near_ties"],
                         "routing_overlap": dict(m["overlap"], random=cfg.top_k * cfg.top_k / cfg.n_experts)}}
    if batch == 1 and out["kernel"] == "decode_token_fused_kernel" and cfg.name.startswith(("C1", "C2")) and \
            cfg.n_layers == stacks.CONFIGS[cfg.name[:2]].n_layers:
        # DRAM traffic of one launch from the ncu summary of a short cut of this workload (a single
        # sequence streams the same number of experts in every layer, so traffic grows with the depth)
        per_layer, src = profile_value(f"dram_bytes_per_layer_{cfg.name[:2].lower()}_batch1_decode_token_fused_kernel")
        out["traffic"] = per_layer * cfg.n_layers if per_layer else None
        out["traffic_source"] = src
    if cfg.cache_slots:
        h2d = (s1["h2d_bytes_demand"] + s1["h2d_bytes_prefetch"] - s0["h2d_bytes_demand"] - s0["h2d_bytes_prefetch"])
        transfer, exposed = run["transfer_ms"], run["exposed_ms"]
        out["cache"] = {
            "slots": cfg.cache_slots, "hits": run["cache_hits"], "misses": run["cache_misses"],
            "hit_rate": run["cache_hits"] / max(run["cache_hits"] + run["cache_misses"], 1),
            "prefetch_issued": run["prefetch_issued"], "prefetch_useful": run["prefetch_useful"],
            "prefetch_wasted": run["prefetch_wasted"], "h2d_gb": h2d / 1e9, "transfer_ms": transfer, "exposed_ms": exposed,
            "hidden_frac": 1.0 - exposed / max(transfer, 1e-9),
            # no more of the transfer time can be hidden than the compute stream is busy: the rest of
            # the step it waits for copies whatever the predictor does (the link is the bound)
            "hidden_bound": min(1.0, max(m["ms"] - exposed, 0.0) / max(transfer, 1e-9)),
            "prefetch_limit": args.prefetch_limit, "prefetch_min_score": args.prefetch_min_score,
            "prefetch_floor": args.prefetch_floor, "mode": args.mode, "inter_layer_gap_us": args.inter_layer_gap_us,
            "copy_throttle": [args.throttle_chunk_kb, args.throttle_gap_us]}
    return out


def make_stack(cfg, batch, dev, args):
    import paper_2606_15453_b200 as P
    flags = ((P.FLAG_NO_DENSE if args.no_dense else 0) | (P.FLAG_NO_FUSED if args.no_fused else 0) |
             (P.FLAG_NO_PERSISTENT if args.no_persistent else 0))
    st = load_stack(cfg, batch, dev, prefetch_limit=args.prefetch_limit, mode=args.mode, flags=flags)
    if args.prefetch_min_score:
        st.set_prefetch_min_score(args.prefetch_min_score)
    if args.predict_threshold != 2:
        st.set_predict_threshold(args.predict_threshold)
    if args.live_counts:
        st.set_replacement_rule(True)
    if args.dense_min_batch and not args.no_dense:
        st.set_dense_min_batch(args.dense_min_batch)
    if args.stage_known_kb >= 0 or args.stage_pred_mb >= 0:
        st.set_onchip_staging(max(args.stage_known_kb, 0) << 10, int(max(args.stage_pred_mb, 0.0) * 1e6))
    if cfg.cache_slots:
        if args.cache_policy != "default" or args.prefetch_floor >= 0:
            window, by_turn = {"default": (16, True) if cfg.n_layers * min(cfg.n_experts, batch * cfg.top_k) > cfg.cache_slots
                               else (0, False), "lru": (0, False), "counts": (16, False), "turn": (16, True)}[args.cache_policy]
            if args.prefetch_floor >= 0 and window == 0:
                window = 16        # the floor is a test on the use counts: it needs a history window
            st.set_cache_policy(window, by_turn, args.prefetch_floor)
        if args.throttle_chunk_kb:
            st.set_copy_throttle(args.throttle_chunk_kb << 10, args.throttle_gap_us)
    return st


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=192)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default="C1", choices=sorted(stacks.CONFIGS))
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling runs)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--ref-layers", type=int, default=2)
    ap.add_argument("--cpu-sample-layers", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the short runs of the other resident configurations that the default run appends")
    ap.add_argument("--prefetch-limit", type=int, default=0, help="offloaded stacks: copies per layer step")
    ap.add_argument("--prefetch-min-score", type=int, default=0,
                    help="offloaded stacks: prefetch only predictions with at least this score")
    ap.add_argument("--prefetch-floor", type=int, default=-1,
                    help="offloaded stacks: a prefetch only takes a slot whose expert has at most this many uses in "
                         "its history window (-1: no such test)")
    ap.add_argument("--cache-policy", default="default", choices=["default", "lru", "counts", "turn"])
    ap.add_argument("--throttle-chunk-kb", type=int, default=0, help="offloaded stacks: expert copies in chunks of this size ...")
    ap.add_argument("--throttle-gap-us", type=int, default=0, help="... with this much idle time after each (link-speed sweep)")
    ap.add_argument("--mode", default="st", choices=["off", "temporal", "spatial", "st"])
    ap.add_argument("--live-counts", action="store_true",
                    help="Algorithm 3 replaces a candidate by the routed expert with the largest live co-activation count")
    ap.add_argument("--predict-threshold", type=int, default=2, help="set threshold of Algorithm 2 (the paper: 2)")
    ap.add_argument("--inter-layer-gap-us", type=float, default=0.0,
                    help="idle the compute stream this long after every layer: a stand-in for the attention "
                         "block the paper overlaps expert prefetch with (Section 4.3.4); 0 = pure MoE stack")
    ap.add_argument("--cache-slots", type=int, default=0,
                    help="offloaded stacks: override the number of HBM slots (a few times top_k: the paper's setting, "
                         "a buffer for one layer's experts and no cache)")
    ap.add_argument("--resident", action="store_true", help="keep every expert in HBM (cache_slots = 0)")
    ap.add_argument("--dense-min-batch", type=int, default=0,
                    help="smallest batch that takes the tcgen05 path (0: the library's default, 2)")
    ap.add_argument("--stage-known-kb", type=int, default=-1,
                    help="three-phase single-sequence kernel: L2 staging of known weights, KiB per expert and SM "
                         "(-1: the library's default, 0: off)")
    ap.add_argument("--stage-pred-mb", type=float, default=-1.0,
                    help="three-phase single-sequence kernel: MB per layer of predicted experts' rows staged into L2 "
                         "ahead of the router (-1: the library's default)")
    ap.add_argument("--no-dense", action="store_true",
                    help="batched steps of resident bf16 stacks on the CUDA-core kernels instead of the tcgen05 ones")
    ap.add_argument("--no-persistent", action="store_true",
                    help="resident stacks: per-layer kernels (replayed as a CUDA graph) instead of one persistent kernel per step")
    ap.add_argument("--no-fused", action="store_true",
                    help="single-sequence resident steps on the three-phase kernel instead of the one-phase one")
    args = ap.parse_args()

    cfg = stacks.CONFIGS[args.workload]
    if args.layers:
        cfg = cfg.scaled(n_layers=args.layers,
                         cache_slots=min(cfg.cache_slots, args.layers * cfg.n_experts))
    if args.resident:
        cfg = cfg.scaled(cache_slots=0, name=cfg.name + "-resident")
    if args.cache_slots:
        cfg = cfg.scaled(cache_slots=args.cache_slots, name=cfg.name + f"-slots{args.cache_slots}")
    batch = args.batch
    if args.impl == "reference":
        return run_reference(args, cfg, batch)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    import paper_2606_15453_b200 as P
    P.build()
    default_run = (args.workload == "C1" and batch == 1 and not args.layers and not args.resident
                   and not args.no_secondary and world == 1)
    # the default run also times C1 at batch 4 on the same 90 GB stack (a full replica per rank)
    st = make_stack(cfg, 4 if default_run else batch, dev, args)
    stream = torch.cuda.Stream()            # a capturable stream: decode steps replay as a CUDA graph
    torch.cuda.set_stream(stream)
    L, K, H = cfg.n_layers, cfg.top_k, cfg.hidden
    m = measure(cfg, batch, st, args, dev, world, stream, with_e2e=True)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    head = summarise(cfg, batch, m, args, world, peak)
    tokens = args.steps * batch * world
    persistent = cfg.cache_slots == 0 and not args.no_persistent   # resident stacks: one kernel launch per decode step
    whole_step = head["kernel"].startswith("decode_token")
    traffic, traffic_src = head.get("traffic"), head.get("traffic_source")
    out = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": workload_config(cfg, batch, world),
        "path": {"ffn_path": {"decode_token_fused_kernel": "row triples (gate, up, transposed down) streamed by bulk "
                                                             "copies into shared memory, CUDA-core FMAs, one phase per layer",
                                "decode_token_kernel": "weight-streaming GEMV on CUDA cores, three phases per layer",
                                "gate_up_kernel": "weight-streaming GEMV on CUDA cores, per-layer kernels"}.get(
                                    head["kernel"], "tcgen05 tiles (TMA-fed, TMEM accumulators)"),
                 "resident_weight_gb": round(L * (cfg.n_experts + cfg.n_shared) * cfg.expert_bytes / 1e9, 1)},
        "clocks": head["clocks"],
        "e2e": {"value": tokens / (m["e2e_ms"] * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": batch * H * 4,
                "d2h_bytes_per_step": batch * H * 4 + L * batch * K * 4},
        "gpu_launches": head["gpu_launches"],
        "roofline": {"bound": "hbm", "kernel": head["kernel"],
                     "achieved": head["achieved_gbs"], "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": head["frac"], "frac_of_8000": head["frac_of_8000"],
                     "traffic": traffic, "traffic_source": traffic_src,
                     "algorithmic_bytes_per_launch": head["algorithmic_bytes_per_step"] if persistent else None,
                     "us_per_launch": head["ms_per_step"] * 1e3 if persistent else None,
                     "note": None if persistent else "offloaded stack: whole-step figures; per-layer kernels, time dominated by "
                                                     "host->HBM expert copies (see cache)"},
        "predictor": head["predictor"],
    }
    if "cache" in head:
        out["cache"] = head["cache"]
    if default_run:
        # short runs of the other resident benchmark configurations, so that the roofline fractions
        # of all of them are in this line (same fields each; `kernel` names what ran)
        sec = []
        short = argparse.Namespace(**{**vars(args), "steps": 48, "warmup": 4})
        try:    # a failure here must not cost the headline line
            sec.append(summarise(cfg, 4, measure(cfg, 4, st, short, dev, world, stream, with_e2e=False), short, world, peak))
            st.close()
            del st
            torch.cuda.empty_cache()
            c2 = stacks.CONFIGS["C2"]
            st2 = make_stack(c2, 8, dev, short)
            for b in (1, 8):
                sec.append(summarise(c2, b, measure(c2, b, st2, short, dev, world, stream, with_e2e=False), short, world, peak))
            st2.close()
            del st2
        except Exception as e:  # noqa: BLE001
            sec.append({"error": repr(e)})
        out["secondary"] = sec
    else:
        st.close()
    torch.cuda.empty_cache()
    if world == 1 and not args.no_cpu_baseline:
        layers = min(L, args.cpu_sample_layers)
        try:
            spent, cores = cpu_oracle_sample(cfg, batch, layers, 2, dev)
            per_token = spent[-1] * L / layers
            out["cpu_baseline"] = {
                "value": batch / per_token, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"second decode step, first {layers} of {L} layers, batch {batch}, "
                          f"scaled to the full depth"}
        except Exception as e:  # noqa: BLE001
            out["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": 0, "kind": "oracle", "sample": "failed: " + repr(e)}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
