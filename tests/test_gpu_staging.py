"""On-chip staging in the single-sequence persistent decode step: hinting known and predicted
weight rows into L2 ahead of the phase that reads them never changes a result, and the
row-slice schedule of that kernel agrees bit for bit with the per-layer kernels."""
import pytest
import torch

import paper_2606_15453_b200 as P
from datagen import stacks
from helpers import Pair

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(cfg, T, flags=0, staging=None):
    pr = Pair(cfg, 1, oracle=False, flags=flags | P.FLAG_NO_FUSED)    # the three-phase kernel family
    if staging is not None:
        pr.stack.set_onchip_staging(*staging)
    L, K = cfg.n_layers, cfg.top_k
    ids = torch.empty(L, 1, K, dtype=torch.int32, device=DEV)
    w = torch.empty(L, 1, K, dtype=torch.float32, device=DEV)
    pred = torch.empty(L, 1, pr.stack.max_pred, dtype=torch.int32, device=DEV)
    npred = torch.empty(L, 1, dtype=torch.int32, device=DEV)
    ho = torch.empty(1, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, 1, T).to(DEV)
    rec = []
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for t in range(T):
            pr.stack.decode_token(x[t].clone(), ho, ids, w, pred, npred, stream=stream)
            stream.synchronize()
            rec.append((ho.cpu().clone(), ids.cpu().clone(), w.cpu().clone(), pred.cpu().clone(), npred.cpu().clone()))
    out = rec, pr.stack.export_state(), pr.stack.stats()
    pr.close()
    return out


@pytest.mark.parametrize("shape", [
    dict(dtype="bf16", hidden=512, inter=352, n_experts=16, top_k=3, n_shared=1),
    dict(dtype="bf16", hidden=272, inter=176, n_experts=33, top_k=4, n_shared=2),   # ragged rows, slices of 1-2 rows
    dict(dtype="fp8", hidden=1024, inter=768, n_experts=32, top_k=8, n_shared=0),
    dict(dtype="f32", hidden=256, inter=64, n_experts=8, top_k=2, n_shared=0),       # fewer rows than SMs
    dict(dtype="bf16", hidden=256, inter=9216, n_experts=8, top_k=2, n_shared=1),    # down rows cut into segments
])
def test_staging_and_schedule_never_change_results(shape):
    cfg = stacks.CONFIGS["C2"].scaled(n_layers=4, profile_tokens=3, cache_slots=0, **shape)
    T = 8
    base = _run(cfg, T, staging=(1 << 20, 0))                   # known weights staged
    assert base[2]["kernel_launches"] <= T + 1                  # one persistent launch per step (+ table build)
    assert base[2]["hits"] > 0 and base[2]["predicted"] > 0
    variants = {
        "off": _run(cfg, T, staging=(0, 0)),
        "predicted": _run(cfg, T, staging=(1 << 20, 8_000_000)),
        "tiny budgets": _run(cfg, T, staging=(4096, 100_000)),
        "per-layer kernels": _run(cfg, T, flags=P.FLAG_NO_PERSISTENT),
    }
    for name, other in variants.items():
        for t, (a, b) in enumerate(zip(base[0], other[0])):
            assert all(torch.equal(u, v) for u, v in zip(a, b)), (name, t)
        assert base[1] == other[1], name                        # predictor tables, byte for byte
    assert variants["per-layer kernels"][2]["kernel_launches"] > base[2]["kernel_launches"]


def test_staging_setter_rejects_bad_arguments():
    cfg = stacks.CONFIGS["C0"].scaled(n_layers=2)
    pr = Pair(cfg, 1, oracle=False)
    with pytest.raises(P.StmoeError):
        pr.stack.set_onchip_staging(-1, 0)
    with pytest.raises(P.StmoeError):
        pr.stack.set_onchip_staging(0, -5)
    pr.close()
