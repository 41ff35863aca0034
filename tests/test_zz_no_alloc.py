"""The allocation-free FFN entry point (stmoe_moe_ffn_static) against stmoe_moe_ffn.

Some hosts cannot allocate device memory while they run (a serving loop where cudaMalloc may
stall the device, a framework that already owns all of HBM); for them the library carries its
own 8 MiB scratch area.  This file is collected last so that a run that stops at the first
failure has already run every other test; it passes alone in a fresh process as well.
"""
import numpy as np
import pytest
import torch

import paper_2606_15453_b200 as P
from datagen import rng, stacks
from helpers import TOL, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _problem(seed, B, E, K, H, I, dt):
    cfg = stacks.CONFIGS["C0"].scaled(hidden=H, inter=I, dtype=dt, n_experts=E, top_k=K)
    nbytes = P.expert_image_bytes(H, I, dt)
    img = torch.zeros(E, nbytes, dtype=torch.uint8, device=DEV)
    for e in range(E):
        w = stacks.expert_weights(cfg, seed, e, device=DEV)
        flat = torch.cat([w[k].contiguous().view(torch.uint8).flatten() for k in ("gate", "up", "down")])
        img[e, :flat.numel()] = flat
    h = rng.normal(B * H, rng.stream_key(90, seed)).view(B, H).to(DEV)
    inv = (1.0 / torch.sqrt((h.double() ** 2).mean(1) + 1e-6)).float()
    sel = torch.argsort(rng.uniform_bits(B * E, rng.stream_key(91, seed)).view(B, E), dim=1)[:, :K]
    ids = torch.sort(sel, dim=1).values.to(torch.int32).to(DEV)
    w = (rng.uniform01(B * K, rng.stream_key(92, seed)).view(B, K) * 0.4 + 0.1).float().to(DEV)
    return img, h, inv, ids, w


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row():
    E, K, H, I, dt = 6, 2, 512, 1408, "bf16"
    scratch = torch.empty(P.moe_ffn_scratch_bytes(5, K, H, I), dtype=torch.uint8, device=DEV)
    for call, B in enumerate((5, 3)):          # second call: other inputs, stale area contents
        img, h, inv, ids, w = _problem(call, B, E, K, H, I, dt)
        want = torch.empty(B, H, device=DEV)
        got = torch.full((B, H), float("nan"), device=DEV)
        P.moe_ffn(h, inv, ids, w, img, dt, E, H, I, 0.1, want, scratch)
        P.moe_ffn_static(h, inv, ids, w, img, dt, E, H, I, 0.1, got)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert rel_err(got.cpu().numpy(), want.cpu().numpy()) <= TOL[dt]
        moe_w, moe_g = (want - h).cpu().numpy() / 0.1, (got - h).cpu().numpy() / 0.1
        assert rel_err(moe_g, moe_w) <= 1e-3


def test_static_scratch_rejects_problems_beyond_its_capacity():
    E, K, H, I = 4, 8, 4096, 14336
    B = 64
    assert P.moe_ffn_scratch_bytes(B, K, H, I) > (8 << 20)
    h = torch.zeros(B, H, device=DEV)
    ids = torch.zeros(B, K, dtype=torch.int32, device=DEV)
    w = torch.zeros(B, K, device=DEV)
    img = torch.zeros(16, dtype=torch.uint8, device=DEV)      # never touched: the call is refused
    with pytest.raises(P.StmoeError, match="capacity"):
        P.moe_ffn_static(h, None, ids, w, img, "bf16", E, H, I, 0.1, torch.empty_like(h))
