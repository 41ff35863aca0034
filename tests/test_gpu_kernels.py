"""GPU parity of the single kernels (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2606_15453_b200 as P
from datagen import rng, stacks
from helpers import TOL, rel_err, scales_blob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_generators_give_identical_bits_on_cpu_and_gpu():
    key = rng.stream_key(0, 11, 3, 5, 1)
    assert torch.equal(rng.normal(300_000, key), rng.normal(300_000, key, device=DEV).cpu())
    for name in ("C0", "C4"):
        cfg = stacks.CONFIGS[name].scaled(hidden=128, inter=208)
        a, b = stacks.expert_weights(cfg, 1, 2), stacks.expert_weights(cfg, 1, 2, device=DEV)
        for k in a:
            assert torch.equal(a[k].view(torch.uint8), b[k].cpu().view(torch.uint8)), (name, k)


@pytest.mark.parametrize("B,E,H,K,dt", [
    (1, 8, 256, 2, "f32"), (4, 8, 4096, 2, "bf16"), (8, 64, 2048, 6, "bf16"),
    (16, 128, 2048, 8, "bf16"), (3, 60, 272, 4, "bf16"), (5, 160, 528, 8, "f32"),
    (2, 256, 1024, 8, "bf16"), (64, 9, 144, 9, "f32"), (1, 33, 48, 1, "bf16")])
def test_router_topk_matches_oracle(B, E, H, K, dt):
    Wf = rng.normal(E * H, rng.stream_key(7, E, H)).view(E, H) * 0.02
    W = Wf if dt == "f32" else Wf.to(torch.bfloat16)
    h = rng.normal(B * H, rng.stream_key(8, B, H)).view(B, H) * 1.7
    if B > 2:   # plant an exact tie across the K-th place in sequence 1
        W = W.clone()
        r = O.route(h[1].numpy(), W.contiguous(), dt, K)
        if K < E:
            order = np.argsort(-r["z"], kind="stable")
            W[order[K]] = W[order[K - 1]]
    W = W.contiguous()
    out = P.router_topk(h.to(DEV), W.to(DEV), K)
    torch.cuda.synchronize()
    for b in range(B):
        r = O.route(h[b].numpy(), W, dt, K)
        z = out["logits"][b].cpu().numpy()
        assert np.abs(z - r["z"]).max() < 2e-5 * max(1.0, np.abs(r["z"]).max())
        _, gap = O.topk(r["z"], K)
        if gap > 1.2e-4:
            assert out["ids"][b].cpu().tolist() == r["ids"].tolist()
            assert np.abs(out["w"][b].cpu().numpy() - r["w"]).max() < 2e-6
            assert int(out["flags"][b]) == 0
        elif gap < 0.8e-4:
            assert int(out["flags"][b]) == 1
        if gap == 0.0:     # exact tie: the lower id must win on both sides
            assert out["ids"][b].cpu().tolist() == r["ids"].tolist()
        assert sorted(out["ids"][b].cpu().tolist()) == out["ids"][b].cpu().tolist()
    assert abs(float(out["inv_rms"][0]) - 1 / np.sqrt(np.mean(h[0].double().numpy() ** 2) + 1e-6)) < 1e-5


def test_router_topk_renorm_and_bad_arguments():
    h = rng.normal(2 * 64, rng.stream_key(1, 1)).view(2, 64).to(DEV)
    W = (rng.normal(8 * 64, rng.stream_key(1, 2)).view(8, 64) * 0.1).to(DEV)
    out = P.router_topk(h, W, 3, renorm=True)
    assert torch.allclose(out["w"].sum(1).cpu(), torch.ones(2), atol=1e-6)
    with pytest.raises(P.StmoeError):
        P.router_topk(h, W, 9)               # K > E
    with pytest.raises(P.StmoeError):
        P.router_topk(h[:, :40].contiguous(), W[:, :40].contiguous(), 2)   # H not a multiple of 16


def _images(cfg, n_experts):
    """Expert images for the stand-alone FFN entry point + CPU copies for the oracle."""
    nbytes = P.expert_image_bytes(cfg.hidden, cfg.inter, cfg.dtype)
    img = torch.zeros(n_experts, nbytes, dtype=torch.uint8, device=DEV)
    cpu = []
    for e in range(n_experts):
        w = stacks.expert_weights(cfg, 0, e, device=DEV)
        parts = [w["gate"], w["up"], w["down"]] + ([scales_blob(w)] if cfg.dtype == "fp8" else [])
        flat = torch.cat([p.contiguous().view(torch.uint8).flatten() for p in parts])
        img[e, :flat.numel()] = flat
        cpu.append({k: v.cpu().contiguous() for k, v in w.items()})
    return img, cpu


@pytest.mark.parametrize("dt,B,E,K,H,I", [
    ("f32", 1, 8, 2, 256, 512), ("bf16", 1, 4, 2, 512, 1408), ("bf16", 5, 3, 2, 272, 176),
    ("fp8", 1, 4, 2, 512, 768), ("fp8", 7, 4, 3, 256, 400), ("f32", 9, 5, 5, 144, 80),
    ("bf16", 4, 8, 2, 4096, 1024), ("bf16", 16, 16, 8, 2048, 768)])
def test_moe_ffn_matches_oracle(dt, B, E, K, H, I):
    cfg = stacks.CONFIGS["C0"].scaled(hidden=H, inter=I, dtype=dt, n_experts=E, top_k=K)
    img, cpu = _images(cfg, E)
    h = rng.normal(B * H, rng.stream_key(21, B, H)).view(B, H)
    inv = (1.0 / torch.sqrt((h.double() ** 2).mean(1) + 1e-6)).float()
    sel = torch.argsort(rng.uniform_bits(B * E, rng.stream_key(22, B, E)).view(B, E), dim=1)[:, :K]
    ids = torch.sort(sel, dim=1).values.to(torch.int32)
    w = (rng.uniform01(B * K, rng.stream_key(23, B)).view(B, K) * 0.5 + 0.05).float()
    scratch = torch.empty(P.moe_ffn_scratch_bytes(B, K, H, I), dtype=torch.uint8, device=DEV)
    out = torch.empty(B, H, dtype=torch.float32, device=DEV)
    P.moe_ffn(h.to(DEV), inv.to(DEV), ids.to(DEV), w.to(DEV), img, dt, E, H, I, 0.1, out, scratch)
    torch.cuda.synchronize()
    for b in range(B):
        x = (h[b] * inv[b]).numpy()
        yk = np.stack([O.expert_ffn(x, cpu[int(e)], dt) for e in ids[b]])
        ref = O.combine(h[b].numpy(), None, yk, w[b].numpy(), 0.1)
        got = out[b].cpu().numpy()
        moe_ref, moe_got = (ref - h[b].numpy()) / 0.1, (got - h[b].numpy()) / 0.1
        assert rel_err(got, ref) <= TOL[dt]
        assert rel_err(moe_got, moe_ref) <= 1e-3, rel_err(moe_got, moe_ref)


def test_moe_ffn_is_reproducible_and_rejects_short_scratch():
    cfg = stacks.CONFIGS["C0"].scaled(hidden=256, inter=512, dtype="bf16", n_experts=4, top_k=2)
    img, _ = _images(cfg, 4)
    h = rng.normal(6 * 256, rng.stream_key(31)).view(6, 256).to(DEV)
    ids = torch.tensor([[0, 1], [1, 2], [0, 3], [1, 3], [0, 1], [2, 3]], dtype=torch.int32, device=DEV)
    w = torch.full((6, 2), 0.3, device=DEV)
    scratch = torch.empty(P.moe_ffn_scratch_bytes(6, 2, 256, 512), dtype=torch.uint8, device=DEV)
    a, b = torch.empty_like(h), torch.empty_like(h)
    P.moe_ffn(h, None, ids, w, img, "bf16", 4, 256, 512, 0.1, a, scratch)
    scratch.fill_(0xAB)   # stale scratch contents must not matter
    P.moe_ffn(h, None, ids, w, img, "bf16", 4, 256, 512, 0.1, b, scratch)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    with pytest.raises(P.StmoeError):
        P.moe_ffn(h, None, ids, w, img, "bf16", 4, 256, 512, 0.1, a, scratch[:1024])
