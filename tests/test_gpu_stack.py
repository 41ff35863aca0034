"""GPU parity of the whole layer step on seeded stacks: teacher-forced layer outputs,
predictor replay on the GPU's own routing, free-running decode, cache bookkeeping."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2606_15453_b200 as P
from datagen import stacks
from helpers import Pair, cache_policy, check_layer

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _teacher_forced(cfg, B, tokens, mode="st", prefetch_limit=0, flags=0, min_score=0):
    """Feed both sides the oracle's hidden state at every (token, layer)."""
    pr = Pair(cfg, B, mode=mode, prefetch_limit=prefetch_limit, flags=flags)
    if min_score:
        pr.stack.set_prefetch_min_score(min_score)
    x = stacks.token_inputs(cfg, B, tokens).numpy()
    replay = O.Predictor(cfg.n_layers, cfg.n_experts, cfg.top_k, B, cfg.profile_tokens, mode)
    cache = O.CacheModel(cfg.cache_slots, cfg.n_layers, cfg.n_experts, **cache_policy(cfg, B)) if cfg.cache_slots else None
    skipped = 0
    for t in range(tokens):
        h = x[t]
        for l in range(cfg.n_layers):
            o = pr.oracle.layer_step(l, h)
            g = pr.gpu_step(l, h)
            skipped += check_layer(cfg, g, o, h, where=f"t={t} l={l}")
            # predictor replay: the oracle's tables driven by the GPU's routing, bit-exact
            rp = replay.step(l, g["ids"])
            assert g["n_pred"].tolist() == rp["n_pred"].tolist(), (t, l)
            assert (g["pred_ids"] == rp["pred_ids"]).all(), (t, l)
            if cache is not None:
                cache.step(l, np.unique(g["ids"]), (l + 1) % cfg.n_layers,
                           rp["queue_ids"][rp["queue_score"] >= min_score],
                           prefetch_limit)
            h = o["h_out"]
    assert pr.stack.export_state() == replay.export()
    st, so = pr.stack.stats(), replay.stats()
    assert (st["runtime_steps"], st["routed"], st["predicted"], st["hits"]) == \
        (so["steps"], so["routed"], so["predicted"], so["hits"])
    if cache is not None:
        sc = cache.stats()
        assert (st["cache_hits"], st["cache_misses"], st["prefetch_issued"], st["prefetch_useful"],
                st["prefetch_wasted"], st["prefetch_dropped"], st["prefetch_resident"]) == \
            (sc["hits"], sc["misses"], sc["pf_issued"], sc["pf_useful"], sc["pf_wasted"],
             sc["pf_dropped"], sc["pf_resident"])
        assert (pr.stack.export_cache_tags().numpy() == cache.tags()).all()
        assert st["h2d_bytes_demand"] == sc["misses"] * P.expert_image_bytes(cfg.hidden, cfg.inter, cfg.dtype)
    pr.close()
    return skipped, st


def test_c0_full_teacher_forced():
    cfg = stacks.CONFIGS["C0"]
    skipped, st = _teacher_forced(cfg, 1, cfg.tokens)
    assert skipped <= 3
    assert st["decode_steps"] == cfg.tokens and st["hits"] > 0


def test_c0_free_running_and_routing_independent_of_predictor():
    """Both sides run their own residual stream; outputs and routing are the same with the
    predictor on or off (prediction never alters routing)."""
    cfg = stacks.CONFIGS["C0"]
    x = stacks.token_inputs(cfg, 1, cfg.tokens)
    outs = {}
    for mode in ("st", "off"):
        pr = Pair(cfg, 1, mode=mode, oracle=(mode == "st"))
        L, K = cfg.n_layers, cfg.top_k
        ids = torch.empty(L, 1, K, dtype=torch.int32, device=DEV)
        ho = torch.empty(1, cfg.hidden, device=DEV)
        all_ids, all_h, first_div = [], [], None
        for t in range(cfg.tokens):
            pr.stack.decode_token(x[t].to(DEV), ho, routed_ids=ids)
            torch.cuda.synchronize()
            all_ids.append(ids.cpu().numpy().copy()), all_h.append(ho.cpu().numpy().copy())
            if mode == "st" and first_div is None:
                h_o, per = pr.oracle.decode_token(x[t].numpy())
                o_ids = np.stack([r["ids"] for r in per])
                ties = sum(int(r["ties"].sum()) for r in per)
                if (o_ids != all_ids[-1]).any():
                    assert ties > 0, f"routing diverged at token {t} without a near tie"
                    first_div = t
                else:
                    assert np.abs(all_h[-1] - h_o).max() / np.abs(h_o).max() < 1e-4
        outs[mode] = (np.stack(all_ids), np.stack(all_h))
        pr.close()
    assert (outs["st"][0] == outs["off"][0]).all() and (outs["st"][1] == outs["off"][1]).all()


@pytest.mark.parametrize("name,B,kw,tokens", [
    ("C1", 1, dict(n_layers=2, profile_tokens=2), 4),
    ("C1", 4, dict(n_layers=2, profile_tokens=1), 3),
    ("C2", 1, dict(n_layers=3, profile_tokens=2), 5),
    ("C2", 8, dict(n_layers=2, profile_tokens=1), 3),
    ("C3", 1, dict(n_layers=3, profile_tokens=2, cache_slots=96), 6),
    ("C3", 16, dict(n_layers=2, profile_tokens=1, cache_slots=160), 3),
    ("C4", 1, dict(n_layers=2, profile_tokens=1, cache_slots=64), 3),
    ("C4", 32, dict(n_layers=2, profile_tokens=1, cache_slots=256, hidden=1024, inter=768), 2),
])
def test_config_shapes_teacher_forced(name, B, kw, tokens):
    """The benchmark shapes (full H/I, fewer layers) incl. shared experts, offload and fp8."""
    cfg = stacks.CONFIGS[name].scaled(**kw)
    _teacher_forced(cfg, B, tokens, prefetch_limit=8 if cfg.cache_slots else 0)


def test_ragged_shapes_and_modes():
    cfg = stacks.CONFIGS["C0"].scaled(n_layers=3, n_experts=12, top_k=3, hidden=272, inter=176,
                                      n_shared=1, profile_tokens=2, dtype="bf16")
    for mode in ("temporal", "spatial"):
        _teacher_forced(cfg, 5, 6, mode=mode)
    _teacher_forced(cfg.scaled(n_layers=1, n_experts=4, top_k=4, n_shared=0), 2, 4)
    _teacher_forced(cfg, 3, 4, flags=P.FLAG_RENORM_TOPK)


def test_tiny_cache_thrashes_but_stays_correct():
    cfg = stacks.CONFIGS["C0"].scaled(n_layers=3, n_experts=16, top_k=2, hidden=128, inter=256,
                                      profile_tokens=3, dtype="bf16", cache_slots=4)
    _, st = _teacher_forced(cfg, 2, 12)
    assert st["cache_misses"] > 0 and st["transfer_ms"] > 0
    _, st = _teacher_forced(cfg.scaled(cache_slots=48), 2, 12, prefetch_limit=2)
    assert st["prefetch_issued"] > 0


@pytest.mark.parametrize("B,shape", [
    (1, dict(hidden=512, inter=352, n_experts=16, top_k=3)),
    (4, dict(hidden=512, inter=352, n_experts=16, top_k=3)),
    (33, dict(hidden=272, inter=208, n_experts=256, top_k=8, n_shared=1)),     # maximum expert count
    (64, dict(hidden=144, inter=96, n_experts=40, top_k=32, n_shared=0)),      # maximum batch and K
])
def test_decode_token_paths_agree(B, shape):
    """decode_token has three execution paths for a resident stack that share their arithmetic:
    the persistent three-phase kernel, per-layer kernels replayed as a CUDA graph (capturable stream), and per-layer
    kernels launched one by one (default stream).  Outputs, routing, predictions, tables and
    counters must be identical, bit for bit."""
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=3, profile_tokens=3, **shape)
    T = 10 if B <= 4 else 5
    x = stacks.token_inputs(cfg, B, T).to(DEV)
    results = []
    for path in ("persistent", "graph", "eager"):
        pr = Pair(cfg, B, oracle=False,
                  flags=P.FLAG_NO_DENSE | P.FLAG_NO_FUSED | (0 if path == "persistent" else P.FLAG_NO_PERSISTENT))
        L, K = cfg.n_layers, cfg.top_k
        ids = torch.empty(L, B, K, dtype=torch.int32, device=DEV)
        w = torch.empty(L, B, K, dtype=torch.float32, device=DEV)
        pred = torch.empty(L, B, pr.stack.max_pred, dtype=torch.int32, device=DEV)
        npred = torch.empty(L, B, dtype=torch.int32, device=DEV)
        h_in, ho = torch.empty(B, cfg.hidden, device=DEV), torch.empty(B, cfg.hidden, device=DEV)
        stream = torch.cuda.Stream() if path == "graph" else torch.cuda.current_stream()
        rec = []
        with torch.cuda.stream(stream):
            for t in range(T):
                h_in.copy_(x[t])
                pr.stack.decode_token(h_in, ho, ids, w, pred, npred, stream=stream)
                stream.synchronize()
                rec.append((ho.cpu().clone(), ids.cpu().clone(), w.cpu().clone(), pred.cpu().clone(),
                            npred.cpu().clone()))
        results.append((rec, pr.stack.export_state(), pr.stack.stats()))
        pr.close()
    ref_rec, ref_state, ref_stats = results[0]
    for rec, state, st in results[1:]:
        for a, b in zip(ref_rec, rec):
            assert all(torch.equal(u, v) for u, v in zip(a, b))
        assert state == ref_state
        for k in ("runtime_steps", "routed", "predicted", "hits", "decode_steps", "near_ties"):
            assert st[k] == ref_stats[k], k
    assert ref_stats["kernel_launches"] < results[1][2]["kernel_launches"]


def test_prefetch_min_score_policy_matches_filtered_oracle_queue():
    """Prefetching only predictions with a score of at least m = the cache model driven by the
    oracle's queue cut at that score; fewer copies are issued than with the whole predicted set."""
    cfg = stacks.CONFIGS["C0"].scaled(cache_slots=12, profile_tokens=6)
    _, all_ = _teacher_forced(cfg, 2, 20)
    _, cut = _teacher_forced(cfg, 2, 20, min_score=5)
    assert 0 < cut["prefetch_issued"] < all_["prefetch_issued"]
    assert cut["hits"] == all_["hits"] and cut["predicted"] == all_["predicted"]   # the predictor itself is untouched


def test_argument_and_state_errors():
    with pytest.raises(P.StmoeError):
        P.Stack(2, 8, 2, 100, 64)                       # H not a multiple of 16
    with pytest.raises(P.StmoeError):
        P.Stack(2, 8, 2, 64, 64, cache_slots=1)         # fewer slots than routed experts
    s = P.Stack(2, 8, 2, 64, 64, dtype="f32")
    h = torch.zeros(1, 64, device=DEV)
    with pytest.raises(P.StmoeError):
        s.decode_step(1, h, h)                          # layer 0 is due
    with pytest.raises(P.StmoeError):
        s.decode_step(0, torch.zeros(2, 64, device=DEV), torch.zeros(2, 64, device=DEV))  # batch > max
    s.close()


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_offloaded_batches_take_the_tensor_core_tiles(dtype):
    """An offloaded stack without shared experts runs batched steps on the tcgen05 kernels, whose tensor
    maps cover the slot store: more launches per layer than the CUDA-core tiles (operand cast, weighted
    sum), the same routing and cache traffic while the routing agrees, outputs within the tolerance."""
    cfg = stacks.CONFIGS["C3"].scaled(n_layers=3, profile_tokens=1, cache_slots=64, hidden=512, inter=384,
                                      n_experts=32, top_k=4, dtype=dtype)
    B, T = 8, 4
    L, K = cfg.n_layers, cfg.top_k
    x = stacks.token_inputs(cfg, B, T).to(DEV)
    runs = []
    for flags in (0, P.FLAG_NO_DENSE):
        pr = Pair(cfg, B, oracle=False, flags=flags, prefetch_limit=2)
        ids = torch.empty(L, B, K, dtype=torch.int32, device=DEV)
        ho = torch.empty(B, cfg.hidden, device=DEV)
        outs = []
        for t in range(T):
            pr.stack.decode_token(x[t].clone(), ho, ids)
            torch.cuda.synchronize()
            outs.append((ho.cpu().clone(), ids.cpu().clone()))
        runs.append((outs, pr.stack.stats()))
        pr.close()
    (dense, sd), (core, sc) = runs
    assert sd["kernel_launches"] > sc["kernel_launches"]
    same = True
    for t, ((hd, idd), (hc, idc)) in enumerate(zip(dense, core)):
        if t == 0:
            assert torch.equal(idd[0], idc[0])                      # layer 0 sees identical inputs
        same = same and torch.equal(idd, idc)
        if same:
            assert (hd - hc).abs().max().item() <= 2e-2 * hc.abs().max().item(), t
    if same:
        assert (sd["cache_hits"], sd["cache_misses"], sd["prefetch_issued"]) == \
            (sc["cache_hits"], sc["cache_misses"], sc["prefetch_issued"])
