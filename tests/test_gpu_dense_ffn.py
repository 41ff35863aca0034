"""Tensor-core expert FFN (many tokens per expert) against the oracle's expert network."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2606_15453_b200 as P
from datagen import rng, stacks

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bf16_round(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).float().numpy()


@pytest.mark.parametrize("m,H,I", [(16, 128, 128), (1, 256, 192), (13, 256, 704), (33, 512, 1408),
                                   (64, 2048, 768), (48, 1024, 1472)])
def test_dense_ffn_matches_oracle(m, H, I):
    cfg = stacks.CONFIGS["C0"].scaled(hidden=H, inter=I, dtype="bf16", n_experts=2, top_k=1)
    w = stacks.expert_weights(cfg, 0, 1, device=DEV)
    img = torch.cat([w[k].contiguous().view(torch.uint8).flatten() for k in ("gate", "up", "down")])
    cpu = {k: v.cpu().contiguous() for k, v in w.items()}
    h = rng.normal(m * H, rng.stream_key(41, m, H)).view(m, H)
    inv = (1.0 / torch.sqrt((h.double() ** 2).mean(1) + 1e-6)).float()
    y, flags = P.expert_ffn_dense(h.to(DEV), inv.to(DEV), img, H, I)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    y = y.cpu().numpy()
    for t in range(m):
        # the kernel rounds its inputs to bf16; the oracle gets the same rounded token
        x = _bf16_round((h[t] * inv[t]).numpy())
        ref = O.expert_ffn(x, cpu, "bf16")
        scale = np.abs(ref).max()
        # one more bf16 rounding (of the gated activations, relative 2^-9 each) sits inside
        assert np.abs(y[t] - ref).max() <= 6e-3 * scale, (t, np.abs(y[t] - ref).max() / scale)


def test_dense_ffn_rejects_bad_shapes():
    img = torch.zeros(3 * 128 * 128 * 2, dtype=torch.uint8, device=DEV)
    with pytest.raises(P.StmoeError):
        P.expert_ffn_dense(torch.zeros(65, 128, device=DEV), None, img, 128, 128)   # more than 64 tokens
    with pytest.raises(P.StmoeError):
        P.expert_ffn_dense(torch.zeros(4, 96, device=DEV), None, img, 96, 128)      # hidden not a multiple of 64
