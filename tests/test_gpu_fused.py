"""The single-sequence decode step with one streaming phase per layer (row triples of gate, up
and transposed down rows; exact fixed-point sums across the GPU): parity with the oracle on
whole decode steps, run-to-run reproducibility, agreement with the three-phase kernel."""
import numpy as np
import pytest
import torch

import paper_2606_15453_b200 as P
from datagen import stacks
from helpers import TOL, Pair, decode_tokens_vs_oracle, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

SHAPES = [
    dict(dtype="f32", hidden=256, inter=512, n_experts=8, top_k=2, n_shared=0),        # units of 64 threads
    dict(dtype="bf16", hidden=512, inter=352, n_experts=16, top_k=3, n_shared=1),      # 64 threads, ragged row blocks
    dict(dtype="bf16", hidden=1024, inter=48, n_experts=33, top_k=4, n_shared=2),      # fewer rows than units
    dict(dtype="bf16", hidden=2048, inter=704, n_experts=64, top_k=6, n_shared=2),     # 256 threads (DeepSeek-V2-Lite width)
    dict(dtype="bf16", hidden=4096, inter=512, n_experts=8, top_k=2, n_shared=0),      # 512 threads (Mixtral width)
    dict(dtype="fp8", hidden=4096, inter=768, n_experts=32, top_k=8, n_shared=0),      # fp8, 256 threads, row and column scales
    dict(dtype="fp8", hidden=1024, inter=320, n_experts=256, top_k=8, n_shared=1),     # maximum expert count, 4 experts per thread
    dict(dtype="bf16", hidden=512, inter=64, n_experts=4, top_k=4, n_shared=0),        # K = E: everything routed
    dict(dtype="fp8", hidden=4096, inter=1008, n_experts=16, top_k=8, n_shared=0),     # fp8 with enough row blocks per unit: blocks of four rows
    dict(dtype="fp8", hidden=1024, inter=3536, n_experts=12, top_k=8, n_shared=1),     # four-row blocks, units of two warps
]


@pytest.mark.parametrize("shape", SHAPES)
def test_fused_decode_steps_match_oracle(shape):
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=3, profile_tokens=2, cache_slots=0, **shape)
    st = decode_tokens_vs_oracle(cfg, 1, 5, min_checked=3)
    assert st["kernel_launches"] <= 5 + 1          # one launch per decode step (+ the table build)
    assert st["decode_steps"] == 5


def _run(cfg, T, flags=0):
    pr = Pair(cfg, 1, oracle=False, flags=flags)
    L, K = cfg.n_layers, cfg.top_k
    ids = torch.empty(L, 1, K, dtype=torch.int32, device=DEV)
    w = torch.empty(L, 1, K, dtype=torch.float32, device=DEV)
    pred = torch.empty(L, 1, pr.stack.max_pred, dtype=torch.int32, device=DEV)
    fl = torch.empty(L, 1, dtype=torch.int32, device=DEV)
    ho = torch.empty(1, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, 1, T).to(DEV)
    rec = []
    for t in range(T):
        pr.stack.decode_token(x[t].clone(), ho, ids, w, pred, None, fl)
        torch.cuda.synchronize()
        rec.append((ho.cpu().clone(), ids.cpu().clone(), w.cpu().clone(), pred.cpu().clone(), fl.cpu().clone()))
    out = rec, pr.stack.export_state(), pr.stack.stats()
    pr.close()
    return out


@pytest.mark.parametrize("shape", [SHAPES[1], SHAPES[3], SHAPES[5], SHAPES[8]])
def test_fused_step_is_reproducible_and_agrees_with_three_phase_kernel(shape):
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=4, profile_tokens=2, cache_slots=0, **shape)
    T = 8
    a, b = _run(cfg, T), _run(cfg, T)
    for u, v in zip(a[0], b[0]):          # sums are exact in fixed point: the order of arrival cannot show
        assert all(torch.equal(p, q) for p, q in zip(u, v))
    assert a[1] == b[1]
    three = _run(cfg, T, flags=P.FLAG_NO_FUSED)
    assert three[2]["kernel_launches"] == a[2]["kernel_launches"]
    for t, (u, v) in enumerate(zip(a[0], three[0])):
        if not torch.equal(u[1], v[1]):   # routing parted: only at a flagged near tie
            assert int(u[4].sum()) + int(v[4].sum()) > 0, t
            break
        # fp8 stacks: the one-phase kernel forms its gate/up dot products from f16 pairs (exact weights,
        # activations and eight-term partial sums rounded to f16): a rounding-level difference
        fp8 = cfg.dtype == "fp8"
        assert rel_err(u[0].numpy(), v[0].numpy()) <= (2e-3 if fp8 else 1e-4), t
        assert np.abs(u[2].numpy() - v[2].numpy()).max() < (2e-5 if fp8 else 2e-6)   # (later layers see that h)
        assert torch.equal(u[3], v[3])
    else:
        assert a[1] == three[1]           # same routing all the way: same predictor tables


def test_shapes_outside_the_fused_kernel_use_the_three_phase_kernel():
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=2, profile_tokens=1, hidden=272, inter=176, n_experts=12, top_k=3,
                                      n_shared=1, dtype="bf16")    # 272 columns: not a whole number of warps per row
    st = decode_tokens_vs_oracle(cfg, 1, 3, min_checked=2)
    assert st["kernel_launches"] <= 3 + 1


@pytest.mark.parametrize("flags,B,threshold,live", [(0, 1, 3, False), (P.FLAG_NO_FUSED, 1, 3, False), (0, 1, 2, True),
                                                    (P.FLAG_NO_FUSED, 1, 2, True), (0, 4, 1, True),
                                                    (P.FLAG_NO_DENSE, 3, 2, True)])
def test_in_kernel_predictors_honour_threshold_and_replacement_rule(flags, B, threshold, live):
    """The persistent kernels run Algorithms 2 and 3 inside the kernel (single-sequence row-triple
    kernel, three-phase kernel, tensor-core kernel for batches): with another set threshold, or with
    replacement by live counts, their predictions and tables equal the oracle predictor's,
    replayed on the GPU's routing."""
    import oracle as O
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=4, profile_tokens=3, cache_slots=0, **SHAPES[1])
    pr = Pair(cfg, B, oracle=False, flags=flags)
    pr.stack.set_predict_threshold(threshold)
    pr.stack.set_replacement_rule(live)
    L, K, T = cfg.n_layers, cfg.top_k, 24
    ids = torch.empty(L, B, K, dtype=torch.int32, device=DEV)
    pred = torch.empty(L, B, pr.stack.max_pred, dtype=torch.int32, device=DEV)
    npred = torch.empty(L, B, dtype=torch.int32, device=DEV)
    ho = torch.empty(B, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, B, T).to(DEV)
    replay = O.Predictor(L, cfg.n_experts, K, B, cfg.profile_tokens, "st", threshold=threshold, live_counts=live)
    for t in range(T):
        pr.stack.decode_token(x[t].clone(), ho, ids, None, pred, npred)
        torch.cuda.synchronize()
        for l in range(L):
            rp = replay.step(l, ids[l].cpu().numpy())
            assert npred[l].cpu().tolist() == rp["n_pred"].tolist(), (t, l)
            assert (pred[l].cpu().numpy() == rp["pred_ids"]).all(), (t, l)
    assert pr.stack.export_state() == replay.export()
    if live:
        assert int(O.parse_state(replay.export())["Co"].sum()) == T * B * K * K * (L - 1)
    pr.close()


@pytest.mark.parametrize("B,slots", [(1, 0), (3, 0), (2, 24)])
def test_decode_token_host_equals_the_device_call(B, slots):
    """The host-buffer entry point (copies in, decode step, copies out, wait) against the
    device-pointer call on a second stack: outputs and routing bit-identical, pinned or pageable;
    resident stacks and an offloaded one."""
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=3, profile_tokens=2, cache_slots=slots, **SHAPES[1])
    a, b = Pair(cfg, B, oracle=False), Pair(cfg, B, oracle=False)
    L, K, T = cfg.n_layers, cfg.top_k, 6
    ids = torch.empty(L, B, K, dtype=torch.int32, device=DEV)
    ho = torch.empty(B, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, B, T)
    out_host = torch.empty(B, cfg.hidden).pin_memory()
    ids_host = torch.empty(L, B, K, dtype=torch.int32)
    for t in range(T):
        a.stack.decode_token(x[t].to(DEV), ho, ids)
        b.stack.decode_token_host(x[t].contiguous(), out_host, ids_host if t % 2 == 0 else None)
        torch.cuda.synchronize()
        assert torch.equal(ho.cpu(), out_host), t
        if t % 2 == 0:
            assert torch.equal(ids.cpu(), ids_host), t
    assert a.stack.export_state() == b.stack.export_state()
    a.close(), b.close()
