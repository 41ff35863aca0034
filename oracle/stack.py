"""Whole-stack harness of the CPU oracle (test infrastructure only).

Runs the decode-time MoE layer step layer by layer in the order of the
pipelined workflow (Section 4.3.4): R (route) -> V (verify + Algorithm 3) and
P (Algorithm 2) -> cache model (miss loading, prefetch) -> Com (expert FFNs,
weighted sum) -> residual update h' = h + r * MoE(RMSNorm(h)).  All arithmetic
is done by the C functions of the oracle; this file only sequences them.
"""
from __future__ import annotations

import numpy as np

import oracle as O


class OracleStack:
    """cfg: any object with the StackConfig fields.  router_w: per-layer [E][H]
    CPU tensors.  experts(layer, expert, shared) -> dict of CPU weight tensors."""

    def __init__(self, cfg, router_w, experts, batch=1, mode="st", profile_tokens=None,
                 cache_slots=None, prefetch_limit=0, renorm=False):
        self.cfg, self.router_w, self.experts = cfg, router_w, experts
        self.B = batch
        P = cfg.profile_tokens if profile_tokens is None else profile_tokens
        self.pred = O.Predictor(cfg.n_layers, cfg.n_experts, cfg.top_k, batch, P, mode)
        slots = cfg.cache_slots if cache_slots is None else cache_slots
        self.cache = O.CacheModel(slots, cfg.n_layers, cfg.n_experts) if slots > 0 else None
        self.prefetch_limit = prefetch_limit
        self.renorm = renorm
        self.near_ties = 0

    def route(self, layer, h):
        """h [B][H] -> list of per-sequence route() results."""
        c = self.cfg
        return [O.route(h[b], self.router_w[layer], c.router_dtype, c.top_k, c.rms_eps,
                        self.renorm) for b in range(h.shape[0])]

    def ffn(self, layer, h, routes):
        """Expert FFNs, weighted sum and residual for every sequence."""
        c = self.cfg
        out = np.empty_like(h)
        cache = {}

        def w(e, shared=False):
            if (e, shared) not in cache:
                cache[(e, shared)] = self.experts(layer, e, shared)
            return cache[(e, shared)]

        for b, r in enumerate(routes):
            ys = [O.expert_ffn(r["x"], w(s, True), c.dtype) for s in range(c.n_shared)]
            yk = [O.expert_ffn(r["x"], w(int(e)), c.dtype) for e in r["ids"]]
            out[b] = O.combine(h[b], np.array(ys) if ys else None, np.array(yk), r["w"],
                               c.residual_scale)
        return out

    def bookkeeping(self, layer, ids):
        """Predictor step and cache model on routed ids [B][K]; returns the predictor output."""
        c = self.cfg
        p = self.pred.step(layer, ids)
        if self.cache is not None:
            U = np.unique(np.asarray(ids, dtype=np.int32))
            p["cache"] = self.cache.step(layer, U, (layer + 1) % c.n_layers, p["queue_ids"],
                                         self.prefetch_limit)
        return p

    def layer_step(self, layer, h):
        """One layer step on h [B][H] fp32.  Returns dict(h_out, ids, w, pred_ids, n_pred, ties)."""
        h = np.ascontiguousarray(h, dtype=np.float32)
        routes = self.route(layer, h)
        ids = np.stack([r["ids"] for r in routes])
        p = self.bookkeeping(layer, ids)
        ties = np.array([r["near_tie"] for r in routes], dtype=np.int32)
        self.near_ties += int(ties.sum())
        return dict(h_out=self.ffn(layer, h, routes), ids=ids,
                    w=np.stack([r["w"] for r in routes]), pred_ids=p["pred_ids"],
                    n_pred=p["n_pred"], ties=ties, queue_ids=p["queue_ids"])

    def decode_token(self, h0):
        """All layers for one decode step; returns (h_L, per-layer results)."""
        h, per_layer = np.ascontiguousarray(h0, dtype=np.float32), []
        for layer in range(self.cfg.n_layers):
            r = self.layer_step(layer, h)
            per_layer.append(r)
            h = r["h_out"]
        return h, per_layer
