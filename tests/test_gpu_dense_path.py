"""Decode steps of resident bf16 stacks on the tensor-core (tcgen05) FFN kernels: parity with
the oracle, agreement with the CUDA-core path, reproducibility."""
import numpy as np
import pytest
import torch

import paper_2606_15453_b200 as P
from datagen import stacks
from helpers import Pair, check_layer

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("B,shape", [
    (4, dict(hidden=512, inter=384, n_experts=8, top_k=2, n_shared=0)),
    (9, dict(hidden=272, inter=208, n_experts=16, top_k=3, n_shared=1)),     # ragged row and column tiles
    (16, dict(hidden=2048, inter=768, n_experts=32, top_k=8, n_shared=0)),
    (64, dict(hidden=256, inter=1408, n_experts=64, top_k=6, n_shared=2)),   # 64 tokens on the shared experts
])
def test_dense_layer_steps_match_oracle(B, shape):
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=3, profile_tokens=2, dtype="bf16", **shape)
    pr = Pair(cfg, B)
    x = stacks.token_inputs(cfg, B, 4).numpy()
    skipped = 0
    for t in range(4):
        h = x[t]
        for l in range(cfg.n_layers):
            o = pr.oracle.layer_step(l, h)
            g = pr.gpu_step(l, h)
            skipped += check_layer(cfg, g, o, h, where=f"t={t} l={l}")
            h = o["h_out"]
    st = pr.stack.stats()      # raises if a bounded wait inside a kernel ran out
    assert st["kernel_launches"] == 4 * cfg.n_layers * 6 + 1   # router, predictor, cast, gate/up, down, sum (+ table build)
    assert skipped <= B
    pr.close()


@pytest.mark.parametrize("B,shape", [
    (4, dict(hidden=512, inter=384, n_experts=8, top_k=2, n_shared=0)),
    (9, dict(hidden=272, inter=208, n_experts=16, top_k=3, n_shared=1)),     # ragged row and column tiles
    (33, dict(hidden=1024, inter=768, n_experts=32, top_k=8, n_shared=0)),
    (64, dict(hidden=256, inter=1536, n_experts=64, top_k=6, n_shared=2)),
])
def test_dense_fp8_layer_steps_match_oracle(B, shape):
    """fp8 weights: e4m3 tiles multiplied as stored against three stacked e5m2 activation planes, row scales
    in the epilogue; batches 33 and 64 run gate/up with a single accumulator buffer."""
    cfg = stacks.CONFIGS["C4"].scaled(n_layers=3, profile_tokens=2, cache_slots=0, **shape)
    pr = Pair(cfg, B)
    x = stacks.token_inputs(cfg, B, 3).numpy()
    skipped = 0
    for t in range(3):
        h = x[t]
        for l in range(cfg.n_layers):
            o = pr.oracle.layer_step(l, h)
            g = pr.gpu_step(l, h)
            skipped += check_layer(cfg, g, o, h, where=f"t={t} l={l}")
            h = o["h_out"]
    st = pr.stack.stats()
    assert st["kernel_launches"] == 3 * cfg.n_layers * 6 + 1
    assert skipped <= B
    pr.close()


@pytest.mark.parametrize("B", [4, 17, 40, 64])
def test_dense_fp8_decode_token_agrees_with_cuda_core_path(B):
    """The persistent kernel (stage ring laid out per phase; one or two accumulator buffers) against the
    per-layer kernels bit for bit, and against the CUDA-core path within the tolerance."""
    cfg = stacks.CONFIGS["C4"].scaled(n_layers=3, profile_tokens=3, cache_slots=0, hidden=512, inter=384,
                                      n_experts=16, top_k=4, n_shared=0)
    T = 5
    one = _run_tokens(cfg, B, T, 0, torch.cuda.Stream())
    graph = _run_tokens(cfg, B, T, P.FLAG_NO_PERSISTENT, torch.cuda.Stream())
    eager = _run_tokens(cfg, B, T, P.FLAG_NO_PERSISTENT, torch.cuda.current_stream())
    core = _run_tokens(cfg, B, T, P.FLAG_NO_DENSE, torch.cuda.Stream())
    for other in (graph, eager):    # persistent kernel, replayed graph, plain launches: bit for bit
        for a, b in zip(one[0], other[0]):
            assert all(torch.equal(u, v) for u, v in zip(a, b))
        assert one[1] == other[1]
    assert one[2]["kernel_launches"] < graph[2]["kernel_launches"]
    assert graph[2]["kernel_launches"] > core[2]["kernel_launches"]
    for t, (a, c) in enumerate(zip(graph[0], core[0])):
        scale = c[0].abs().max().item()
        assert (a[0] - c[0]).abs().max().item() <= 2e-2 * scale, t
        if t == 0:
            assert torch.equal(a[1][0], c[1][0])


def _run_tokens(cfg, B, T, flags, stream, min_batch=None):
    pr = Pair(cfg, B, oracle=False, flags=flags)
    if min_batch is not None:
        pr.stack.set_dense_min_batch(min_batch)
    L, K = cfg.n_layers, cfg.top_k
    ids = torch.empty(L, B, K, dtype=torch.int32, device=DEV)
    w = torch.empty(L, B, K, dtype=torch.float32, device=DEV)
    h_in, ho = torch.empty(B, cfg.hidden, device=DEV), torch.empty(B, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, B, T).to(DEV)
    rec = []
    with torch.cuda.stream(stream):
        for t in range(T):
            h_in.copy_(x[t])
            pr.stack.decode_token(h_in, ho, ids, w, stream=stream)
            stream.synchronize()
            rec.append((ho.cpu().clone(), ids.cpu().clone(), w.cpu().clone()))
    out = rec, pr.stack.export_state(), pr.stack.stats()
    pr.close()
    return out


@pytest.mark.parametrize("B", [2, 8, 33])
def test_dense_decode_token_agrees_with_cuda_core_path(B):
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=3, profile_tokens=3, hidden=512, inter=352, n_experts=16,
                                      top_k=3, n_shared=1)
    T = 6
    one = _run_tokens(cfg, B, T, 0, torch.cuda.Stream(), min_batch=2)
    graph = _run_tokens(cfg, B, T, P.FLAG_NO_PERSISTENT, torch.cuda.Stream(), min_batch=2)
    eager = _run_tokens(cfg, B, T, P.FLAG_NO_PERSISTENT, torch.cuda.current_stream(), min_batch=2)
    core = _run_tokens(cfg, B, T, P.FLAG_NO_DENSE, torch.cuda.Stream())
    # the tensor-core path as one persistent kernel, as a replayed graph of per-layer kernels and
    # as plain launches: identical bit for bit
    for other in (graph, eager):
        for a, b in zip(one[0], other[0]):
            assert all(torch.equal(u, v) for u, v in zip(a, b))
        assert one[1] == other[1]
    assert one[2]["kernel_launches"] < graph[2]["kernel_launches"]
    assert graph[2]["kernel_launches"] > core[2]["kernel_launches"]   # per-layer kernels, not the CUDA-core persistent one
    # against the CUDA-core path: same routing while the hidden states stay close (bf16 rounding of
    # the activations moves them a little, so only the first steps are compared id for id)
    for t, (a, c) in enumerate(zip(graph[0], core[0])):
        scale = c[0].abs().max().item()
        assert (a[0] - c[0]).abs().max().item() <= 2e-2 * scale, t
        if t == 0:
            assert torch.equal(a[1][0], c[1][0])      # layer 0 routing sees identical inputs


def test_dense_paths_agree_at_maximum_batch_and_k():
    """64 sequences x top-32: the work list takes 65 KB of the persistent kernel's shared memory and
    leaves a single stage for the ring."""
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=2, profile_tokens=2, hidden=144, inter=96, n_experts=40, top_k=32,
                                      n_shared=0)
    one = _run_tokens(cfg, 64, 4, 0, torch.cuda.Stream())
    graph = _run_tokens(cfg, 64, 4, P.FLAG_NO_PERSISTENT, torch.cuda.Stream())
    core = _run_tokens(cfg, 64, 4, P.FLAG_NO_DENSE, torch.cuda.Stream())
    for a, b in zip(one[0], graph[0]):
        assert all(torch.equal(u, v) for u, v in zip(a, b))
    assert one[1] == graph[1]
    assert one[2]["kernel_launches"] < graph[2]["kernel_launches"]
    for a, c in zip(one[0][:1], core[0][:1]):
        assert torch.equal(a[1][0], c[1][0])
        assert (a[0] - c[0]).abs().max().item() <= 2e-2 * c[0].abs().max().item()


def test_dense_path_off_for_small_batches_and_fp32():
    cfg = stacks.CONFIGS["C0"].scaled(n_layers=2)
    pr = Pair(cfg, 8, oracle=False)        # fp32 weights: no tensor-core path
    with pytest.raises(P.StmoeError):
        pr.stack.set_dense_min_batch(2)
    pr.close()
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=2, hidden=256, inter=256, n_experts=8, top_k=2, n_shared=0)
    pr = Pair(cfg, 8, oracle=False)
    with pytest.raises(P.StmoeError):
        pr.stack.set_dense_min_batch(1)
    pr.close()
