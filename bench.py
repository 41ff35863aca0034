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
# dram__bytes_read.sum + dram__bytes_write.sum of one decode_token_kernel launch, from the ncu
# capture summarised in profiles/decode_token_kernel_c1_2layers_ncu_full.md.  The capture ran a
# 2-layer stack of the same shape (1409.598 MB read + 4.767 MB written); traffic grows in
# proportion to the layer count, so the full launch is that figure x layers / 2.
NCU_TRAFFIC_BYTES_PER_LAYER = {"C1": (1409598000 + 4766976) / 2}


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
        "config": {"workload": cfg.name, "batch": batch, "layers": cfg.n_layers,
                   "experts": cfg.n_experts, "top_k": cfg.top_k, "hidden": cfg.hidden,
                   "inter": cfg.inter},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


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
    ap.add_argument("--prefetch-limit", type=int, default=0, help="offloaded stacks: copies per layer step")
    ap.add_argument("--prefetch-min-score", type=int, default=0,
                    help="offloaded stacks: prefetch only predictions with at least this score")
    ap.add_argument("--mode", default="st", choices=["off", "temporal", "spatial", "st"])
    ap.add_argument("--inter-layer-gap-us", type=float, default=0.0,
                    help="idle the compute stream this long after every layer: a stand-in for the attention "
                         "block the paper overlaps expert prefetch with (Section 4.3.4); 0 = pure MoE stack")
    ap.add_argument("--resident", action="store_true", help="keep every expert in HBM (cache_slots = 0)")
    ap.add_argument("--dense-min-batch", type=int, default=0,
                    help="smallest batch that takes the tcgen05 path (0: the library's default, 2 for bf16, 3 for fp8)")
    ap.add_argument("--stage-known-kb", type=int, default=-1,
                    help="single-sequence resident steps: L2 staging of known weights, KiB per expert and SM "
                         "(-1: the library's default, 0: off)")
    ap.add_argument("--stage-pred-mb", type=float, default=-1.0,
                    help="single-sequence resident steps: MB per layer of predicted experts' rows staged into L2 "
                         "ahead of the router (-1: the library's default)")
    ap.add_argument("--no-dense", action="store_true",
                    help="batched steps of resident bf16 stacks on the CUDA-core kernels instead of the tcgen05 ones")
    args = ap.parse_args()

    cfg = stacks.CONFIGS[args.workload]
    if args.layers:
        cfg = cfg.scaled(n_layers=args.layers,
                         cache_slots=min(cfg.cache_slots, args.layers * cfg.n_experts))
    if args.resident:
        cfg = cfg.scaled(cache_slots=0, name=cfg.name + "-resident")
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
    import paper_2606_15453_b200 as P
    st = load_stack(cfg, batch, dev, prefetch_limit=args.prefetch_limit, mode=args.mode,
                    flags=P.FLAG_NO_DENSE if args.no_dense else 0)  # a full replica per rank
    if args.prefetch_min_score:
        st.set_prefetch_min_score(args.prefetch_min_score)
    if args.dense_min_batch and not args.no_dense:
        st.set_dense_min_batch(args.dense_min_batch)
    if args.stage_known_kb >= 0 or args.stage_pred_mb >= 0:
        st.set_onchip_staging(max(args.stage_known_kb, 0) << 10,
                              int(max(args.stage_pred_mb, 0.0) * 1e6))
    L, K, H = cfg.n_layers, cfg.top_k, cfg.hidden
    n_tok = cfg.profile_tokens + args.warmup + args.steps
    x_host = stacks.token_inputs(cfg, batch, n_tok).pin_memory()
    x_dev = x_host.to(dev)
    h_out = torch.empty(batch, H, device=dev)
    ids = torch.empty(L, batch, K, dtype=torch.int32, device=dev)
    pred = torch.empty(L, batch, st.max_pred, dtype=torch.int32, device=dev)
    npred = torch.empty(L, batch, dtype=torch.int32, device=dev)
    stream = torch.cuda.Stream()            # a capturable stream: decode steps replay as a CUDA graph
    torch.cuda.set_stream(stream)
    h_in = torch.empty(batch, H, device=dev)

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

    # set-up: the profiling phase of Algorithm 1, then warm-up
    t = 0
    for _ in range(cfg.profile_tokens + args.warmup):
        decode(x_dev[t])
        t += 1
    s0 = st.stats()

    # ---- timed region: K decode steps, inputs resident in HBM --------------------------------
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ids_seen = []
    ev0.record(stream)
    for i in range(args.steps):
        decode(x_dev[t + i])
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    s1 = st.stats()

    # ---- same steps again with the FFN kernels bracketed by events (roofline of the top kernel)
    st.set_kernel_timing(True)
    for i in range(args.steps):
        h_in.copy_(x_dev[t + i])
        st.decode_token(h_in, h_out, ids, None, pred, npred)
        ids_seen.append(ids.cpu().numpy().copy())
    st.set_kernel_timing(False)
    s2 = st.stats()

    # ---- end to end: pinned host input copied in, results copied out, every step -------------
    out_host = torch.empty(batch, H).pin_memory()
    ids_host = torch.empty(L, batch, K, dtype=torch.int32).pin_memory()
    barrier()
    w0 = time.perf_counter()
    for i in range(args.steps):
        h_in.copy_(x_host[t + i], non_blocking=True)
        st.decode_token(h_in, h_out, ids, None, pred, npred)
        out_host.copy_(h_out, non_blocking=True)
        ids_host.copy_(ids, non_blocking=True)
        torch.cuda.synchronize()
    e2e_s = time.perf_counter() - w0
    barrier()

    times = torch.tensor([ms, e2e_s * 1e3], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms, e2e_ms = (float(v) for v in times.cpu())
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens = args.steps * batch * world
    value = tokens / (ms * 1e-3)
    peak, peak_kind = measured_peaks()
    step_bytes = [algorithmic_bytes(cfg, a) for a in ids_seen]
    n_ffn = s2["timed_ffn_launches"]
    gate_up_bytes = sum(sum((len(np.unique(a[l])) + cfg.n_shared) for l in range(L)) for a in ids_seen) \
        * (2 * cfg.expert_bytes // 3) / max(n_ffn, 1)
    gu_ms = s2["gate_up_ms"] / max(n_ffn, 1)
    dn_ms = s2["down_ms"] / max(n_ffn, 1)
    achieved = gate_up_bytes / (gu_ms * 1e-3) / 1e9 if gu_ms > 0 else None
    run = {k: s1[k] - s0[k] for k in ("runtime_steps", "routed", "predicted", "hits", "near_ties",
                                      "cache_hits", "cache_misses", "kernel_launches")}
    step_gbs = statistics.mean(step_bytes) / (ms / args.steps * 1e-3) / 1e9
    persistent = cfg.cache_slots == 0          # resident stacks: one kernel launch per decode step
    # batched steps of resident bf16 stacks: expert FFN on tcgen05 tiles (the library's default threshold)
    dense = persistent and not args.no_dense and (
        (cfg.dtype == "bf16" and batch >= (args.dense_min_batch or 2)) or
        (cfg.dtype == "fp8" and batch >= (args.dense_min_batch or 3)))
    top_kernel = "gate_up_kernel"
    if persistent:
        top_kernel = "decode_token_kernel"
        if dense:   # bf16 and fp8: one persistent kernel with the tcgen05 phases
            top_kernel = "decode_token_dense_kernel"
            if cfg.dtype == "fp8" and batch > 4:   # larger fp8 batches: per-layer tcgen05 kernels replayed as a graph
                top_kernel = "dense8_group_kernel<2>"
    whole_step = top_kernel.startswith("decode_token")   # the top kernel is one launch per decode step
    per_layer = NCU_TRAFFIC_BYTES_PER_LAYER.get(args.workload) if batch == 1 else None
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "batch": batch, "layers": L, "experts": cfg.n_experts,
                   "top_k": K, "hidden": H, "inter": cfg.inter, "parallelism": f"replicas x{world}",
                   "profile_tokens": cfg.profile_tokens, "l2": "inputs_larger_than_l2",
                   "ffn_path": "tcgen05 tiles (TMA-fed, TMEM accumulators)" if dense else "weight-streaming GEMV on CUDA cores",
                   "resident_weight_gb": round(L * (cfg.n_experts + cfg.n_shared) * cfg.expert_bytes / 1e9, 1)},
        "clocks": clocks,
        "e2e": {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": batch * H * 4,
                "d2h_bytes_per_step": batch * H * 4 + L * batch * K * 4},
        "gpu_launches": run["kernel_launches"],
        "roofline": {"bound": "hbm",
                     "kernel": top_kernel,
                     "achieved": step_gbs if whole_step else achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": (step_gbs if whole_step else achieved or 0.0) / peak,
                     "frac_of_8000": (step_gbs if whole_step else achieved or 0.0) / 8000.0,
                     "traffic": per_layer * L if (whole_step and per_layer) else None,
                     "algorithmic_bytes_per_launch": statistics.mean(step_bytes) if whole_step else gate_up_bytes,
                     "us_per_launch": ms / args.steps * 1e3 if whole_step else gu_ms * 1e3,
                     "per_layer_kernels": {
                         "note": "second pass over the same steps as per-layer kernels, events around each",
                         "gate_up": {"achieved": achieved, "us_per_launch": gu_ms * 1e3,
                                     "algorithmic_bytes_per_launch": gate_up_bytes},
                         "down": {"achieved": (gate_up_bytes / 2) / (dn_ms * 1e-3) / 1e9 if dn_ms else None,
                                  "us_per_launch": dn_ms * 1e3},
                         "router": {"us_per_launch": s2["router_ms"] / max(n_ffn, 1) * 1e3}},
                     "whole_step": {"bytes_per_token": statistics.mean(step_bytes) / batch,
                                    "achieved": step_gbs, "frac": step_gbs / peak,
                                    "frac_of_8000": step_gbs / 8000.0}},
        "predictor": {"recall": run["hits"] / max(run["routed"], 1),
                      "precision": run["hits"] / max(run["predicted"], 1),
                      "mean_predicted": run["predicted"] / max(run["runtime_steps"], 1),
                      "near_ties": run["near_ties"]},
        "cache": {"slots": cfg.cache_slots, "hits": run["cache_hits"], "misses": run["cache_misses"],
                  "hit_rate": run["cache_hits"] / max(run["cache_hits"] + run["cache_misses"], 1),
                  "prefetch_issued": s1["prefetch_issued"] - s0["prefetch_issued"],
                  "prefetch_useful": s1["prefetch_useful"] - s0["prefetch_useful"],
                  "prefetch_wasted": s1["prefetch_wasted"] - s0["prefetch_wasted"],
                  "h2d_gb": (s1["h2d_bytes_demand"] + s1["h2d_bytes_prefetch"]
                             - s0["h2d_bytes_demand"] - s0["h2d_bytes_prefetch"]) / 1e9,
                  "transfer_ms": s1["transfer_ms"] - s0["transfer_ms"],
                  "exposed_ms": s1["exposed_ms"] - s0["exposed_ms"],
                  "hidden_frac": 1.0 - (s1["exposed_ms"] - s0["exposed_ms"])
                  / max(s1["transfer_ms"] - s0["transfer_ms"], 1e-9),
                  "prefetch_limit": args.prefetch_limit, "prefetch_min_score": args.prefetch_min_score,
                  "mode": args.mode,
                  "inter_layer_gap_us": args.inter_layer_gap_us},
    }
    if world == 1 and not args.no_cpu_baseline:
        st.close()
        torch.cuda.empty_cache()
        layers = min(L, args.cpu_sample_layers)
        spent, cores = cpu_oracle_sample(cfg, batch, layers, 2, dev)
        per_token = spent[-1] * L / layers
        out["cpu_baseline"] = {
            "value": batch / per_token, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"second decode step, first {layers} of {L} layers, batch {batch}, "
                      f"scaled to the full depth"}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
