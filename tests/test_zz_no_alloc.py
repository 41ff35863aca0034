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
        # the two entry points run the same kernels on the same inputs in the same fixed summation
        # order, so the results must agree bit for bit; a tolerance would hide a slip in the layout
        # of the built-in area that disturbs a single partial sum
        assert torch.equal(got, want)


def test_static_entry_point_allocates_no_device_memory():
    """What the entry point is for: after its first call on the device (module load, address
    look-up) further calls, at several problem sizes, leave the device's free memory and the
    caching allocator's reservations exactly as they were."""
    E, K, H, I, dt = 6, 2, 512, 1408, "bf16"
    problems = [_problem(7 + i, B, E, K, H, I, dt) for i, B in enumerate((1, 4, 9, 2))]
    outs = [torch.empty(B, H, device=DEV) for B in (1, 4, 9, 2)]
    img, h, inv, ids, w = problems[0]
    P.moe_ffn_static(h, inv, ids, w, img, dt, E, H, I, 0.1, outs[0])      # first call: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    reserved0, mallocs0 = torch.cuda.memory_reserved(), torch.cuda.memory_stats()["allocation.all.allocated"]
    for _ in range(3):
        for (img, h, inv, ids, w), out in zip(problems, outs):
            P.moe_ffn_static(h, inv, ids, w, img, dt, E, H, I, 0.1, out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    # nothing went through torch's caching allocator either (no segment reserved, no block handed out)
    assert torch.cuda.memory_reserved() == reserved0
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == mallocs0


def test_static_entry_point_reports_malformed_calls_as_bad_arguments():
    h = torch.zeros(1, 520, device=DEV)
    ids = torch.zeros(1, 2, dtype=torch.int32, device=DEV)
    w = torch.zeros(1, 2, device=DEV)
    img = torch.zeros(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(P.StmoeError, match="bad argument"):            # hidden not a multiple of 16
        P.moe_ffn_static(h, None, ids, w, img, "bf16", 4, 520, 64, 0.1, torch.empty_like(h))


def test_static_scratch_rejects_problems_beyond_its_capacity():
    E, K, H, I = 8, 8, 4096, 14336
    B = 64
    assert P.moe_ffn_scratch_bytes(B, K, H, I) > (8 << 20)
    h = torch.zeros(B, H, device=DEV)
    ids = torch.zeros(B, K, dtype=torch.int32, device=DEV)
    w = torch.zeros(B, K, device=DEV)
    img = torch.zeros(16, dtype=torch.uint8, device=DEV)      # never touched: the call is refused
    with pytest.raises(P.StmoeError, match="capacity"):
        P.moe_ffn_static(h, None, ids, w, img, "bf16", E, H, I, 0.1, torch.empty_like(h))
