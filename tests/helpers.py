"""Shared test helpers: build a CUDA stack and the matching oracle from one seeded config."""
import numpy as np
import torch

import oracle as O
import paper_2606_15453_b200 as P
from datagen import stacks
from oracle.stack import OracleStack

TOL = {"f32": 1e-4, "bf16": 2e-2, "fp8": 5e-2}   # max|err| / ||ref||_inf


def cache_policy(cfg, batch):
    """The slot-cache policy the library picks by default: plain LRU unless a decode step can touch
    more (layer, expert) keys than there are slots, then a 16-step use window and the turn order."""
    cyclic = cfg.n_layers * min(cfg.n_experts, batch * cfg.top_k) > cfg.cache_slots
    return dict(window=16 if cyclic else 0, by_turn=cyclic)


def rel_err(got, ref):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30))


def scales_blob(w):
    return torch.cat([w["gate_scale"], w["up_scale"], w["down_scale"]]).contiguous()


class Pair:
    """One seeded stack on both sides.  Expert weights are generated on the GPU once, loaded
    into the CUDA stack and handed (as CPU copies of the same bits) to the oracle on demand."""

    def __init__(self, cfg, batch, mode="st", prefetch_limit=0, flags=0, oracle=True):
        self.cfg, self.B = cfg, batch
        self.dev = torch.device("cuda:0")
        self.router = stacks.router_weights(cfg)
        self.stack = P.Stack.from_config(cfg, max_batch=batch, mode=mode,
                                         prefetch_limit=prefetch_limit, flags=flags)
        self._cpu = {}
        for l in range(cfg.n_layers):
            self.stack.load_router(l, self.router[l])
            for e in range(cfg.n_experts):
                self._load(l, e, False)
            for e in range(cfg.n_shared):
                self._load(l, e, True)
        self.oracle = OracleStack(cfg, self.router, self.experts, batch=batch, mode=mode,
                                  prefetch_limit=prefetch_limit,
                                  renorm=bool(flags & P.FLAG_RENORM_TOPK)) if oracle else None
        K = cfg.top_k
        self.ids = torch.empty(batch, K, dtype=torch.int32, device=self.dev)
        self.w = torch.empty(batch, K, dtype=torch.float32, device=self.dev)
        self.pred = torch.empty(batch, self.stack.max_pred, dtype=torch.int32, device=self.dev)
        self.npred = torch.empty(batch, dtype=torch.int32, device=self.dev)
        self.flags = torch.empty(batch, dtype=torch.int32, device=self.dev)
        self.h_out = torch.empty(batch, cfg.hidden, dtype=torch.float32, device=self.dev)

    def _load(self, l, e, shared):
        w = stacks.expert_weights(self.cfg, l, e, shared, device=self.dev)
        sc = scales_blob(w) if self.cfg.dtype == "fp8" else None
        self.stack.load_experts(l, e, w["gate"], w["up"], w["down"], sc, shared)
        self._gpu_last = w

    def experts(self, layer, expert, shared=False):
        key = (layer, expert, shared)
        if key not in self._cpu:
            w = stacks.expert_weights(self.cfg, layer, expert, shared, device=self.dev)
            self._cpu[key] = {k: v.cpu().contiguous() for k, v in w.items()}
        return self._cpu[key]

    def gpu_step(self, layer, h):
        """h: numpy [B][H] -> dict of numpy results of one stmoe_decode_step."""
        hd = torch.from_numpy(np.ascontiguousarray(h, dtype=np.float32)).to(self.dev)
        self.stack.decode_step(layer, hd, self.h_out, self.ids, self.w, self.pred, self.npred,
                               self.flags)
        torch.cuda.synchronize()
        return dict(h_out=self.h_out.cpu().numpy(), ids=self.ids.cpu().numpy(),
                    w=self.w.cpu().numpy(), pred_ids=self.pred.cpu().numpy(),
                    n_pred=self.npred.cpu().numpy(), ties=self.flags.cpu().numpy() & 1)

    def close(self):
        self.stack.close()


def check_layer(cfg, g, o, h_in, where=""):
    """Compare one layer step: ids exact unless the oracle flags a near tie, weights and output
    within tolerance.  Returns the number of sequences skipped because of a near tie."""
    skipped = 0
    tol = TOL[cfg.dtype]
    for b in range(o["ids"].shape[0]):
        if o["ties"][b] or g["ties"][b]:
            skipped += 1
            if (g["ids"][b] != o["ids"][b]).any():
                continue
        assert (g["ids"][b] == o["ids"][b]).all(), f"{where} b={b}: ids {g['ids'][b]} vs {o['ids'][b]}"
        assert np.abs(g["w"][b] - o["w"][b]).max() < 2e-5, f"{where} b={b}: gate weights"
        moe_g = (g["h_out"][b] - h_in[b]) / cfg.residual_scale
        moe_o = (o["h_out"][b] - h_in[b]) / cfg.residual_scale
        assert rel_err(g["h_out"][b], o["h_out"][b]) <= tol, f"{where} b={b}: layer output"
        assert rel_err(moe_g, moe_o) <= max(tol, 2e-3), f"{where} b={b}: MoE term {rel_err(moe_g, moe_o)}"
    return skipped


def replay_predictor(cfg, batch, mode, trace_ids):
    """Drive the oracle predictor with a routed-id trace [(layer, ids[B][K]) ...]."""
    p = O.Predictor(cfg.n_layers, cfg.n_experts, cfg.top_k, batch, cfg.profile_tokens, mode)
    return p, [p.step(layer, ids) for layer, ids in trace_ids]


def decode_tokens_vs_oracle(cfg, B, T, min_checked, flags=0):
    """Whole decode steps through stmoe_decode_token (the persistent kernels) against the oracle
    running its own residual stream; a sequence is compared while its routing agrees in every
    layer (a disagreement needs a flagged near tie).  The predictor is replayed on the GPU's
    routing, bit-exact.  Returns the stack's statistics."""
    pr = Pair(cfg, B, flags=flags)
    L, K = cfg.n_layers, cfg.top_k
    x = stacks.token_inputs(cfg, B, T)
    ids = torch.empty(L, B, K, dtype=torch.int32, device=pr.dev)
    w = torch.empty(L, B, K, dtype=torch.float32, device=pr.dev)
    pred = torch.empty(L, B, pr.stack.max_pred, dtype=torch.int32, device=pr.dev)
    npred = torch.empty(L, B, dtype=torch.int32, device=pr.dev)
    flags = torch.empty(L, B, dtype=torch.int32, device=pr.dev)   # (the stack's flags were consumed above)
    ho = torch.empty(B, cfg.hidden, device=pr.dev)
    replay = O.Predictor(L, cfg.n_experts, K, B, cfg.profile_tokens, "st")
    checked = 0
    for t in range(T):
        pr.stack.decode_token(x[t].to(pr.dev), ho, ids, w, pred, npred, flags)
        torch.cuda.synchronize()
        g_ids, g_w = ids.cpu().numpy(), w.cpu().numpy()
        for l in range(L):
            rp = replay.step(l, g_ids[l])
            assert npred[l].cpu().tolist() == rp["n_pred"].tolist(), (t, l)
            assert (pred[l].cpu().numpy() == rp["pred_ids"]).all(), (t, l)
        h_ref, per = pr.oracle.decode_token(x[t].numpy())
        o_ids = np.stack([r["ids"] for r in per])
        o_w = np.stack([r["w"] for r in per])
        got = ho.cpu().numpy()
        for b in range(B):
            if (o_ids[:, b] != g_ids[:, b]).any():
                assert sum(int(r["ties"][b]) for r in per) + int(flags[:, b].sum()) > 0, \
                    f"t={t} sequence {b}: routing diverged from the oracle without a near tie"
                continue
            assert np.abs(g_w[0, b] - o_w[0, b]).max() < 2e-5          # layer 0 sees identical inputs
            assert rel_err(got[b], h_ref[b]) <= TOL[cfg.dtype], (t, b)
            xin = x[t][b].numpy()
            assert rel_err(got[b] - xin, h_ref[b] - xin) <= TOL[cfg.dtype], (t, b)
            checked += 1
    assert pr.stack.export_state() == replay.export()
    assert checked >= min_checked
    st = pr.stack.stats()            # raises if a bounded wait inside a kernel ran out
    pr.close()
    return st
