"""The seeded generators: determinism, distribution, planted structure."""
import math

import numpy as np
import torch

from datagen import rng, stacks


def test_normal_is_deterministic_chunk_independent_and_standard():
    key = rng.stream_key(0, 1, 2, 3)
    a = rng.normal(200_000, key)
    b = rng.normal(200_000, key, chunk=4096)
    assert torch.equal(a, b)
    assert torch.equal(a[1000:2000], rng.normal(1000, key, offset=1000))
    assert abs(float(a.mean())) < 0.01 and abs(float(a.std()) - 1.0) < 0.01
    assert abs(float((a.abs() < 1).float().mean()) - 0.6827) < 0.005
    assert not torch.equal(a, rng.normal(200_000, rng.stream_key(0, 1, 2, 4)))


def test_expert_weights_shapes_dtypes_and_scale():
    cfg = stacks.CONFIGS["C0"]
    w = stacks.expert_weights(cfg, 1, 3)
    assert w["gate"].shape == (512, 256) and w["down"].shape == (256, 512)
    assert w["gate"].dtype == torch.float32
    assert abs(float(w["up"].std()) - 0.02) < 0.001
    assert not torch.equal(w["gate"], w["up"])
    c4 = stacks.CONFIGS["C4"].scaled(hidden=64, inter=96)
    w8 = stacks.expert_weights(c4, 0, 0)
    assert w8["gate"].dtype == torch.float8_e4m3fn and w8["gate_scale"].dtype == torch.bfloat16
    deq = w8["down"].float() * w8["down_scale"].float()[:, None]
    assert abs(float(deq.std()) - 0.02) < 0.002
    assert torch.isfinite(w8["gate"].float()).all()


def test_router_chain_correlation():
    cfg = stacks.CONFIGS["C0"]
    ws = [w.double().flatten() for w in stacks.router_weights(cfg)]
    for a, b in zip(ws, ws[1:]):
        r = float(torch.corrcoef(torch.stack([a, b]))[0, 1])
        assert abs(r - 0.8) < 0.05


def test_token_stream_unit_rms_and_ar1():
    cfg = stacks.CONFIGS["C0"]
    x = stacks.token_inputs(cfg, 2, 200).double()
    rms = x.pow(2).mean(-1).sqrt()
    assert abs(float(rms[0].mean()) - 1.0) < 1e-6 and abs(float(rms.mean()) - 1.0) < 0.1
    a, b = x[:-1, 0].flatten(), x[1:, 0].flatten()
    assert abs(float(torch.corrcoef(torch.stack([a, b]))[0, 1]) - cfg.rho) < 0.03
    assert not torch.equal(x[:, 0], x[:, 1])


def test_planted_trace_rate():
    e, f, pi = stacks.planted_pair_trace(8, 0.7, 20000, stream=1)
    assert sorted(pi.tolist()) == list(range(8))
    assert abs(float((f == pi[e]).double().mean()) - 0.7) < 0.01
    assert abs(float(np.bincount(e.numpy(), minlength=8).std()) / 2500) < 0.05


def test_config_sizes():
    c = stacks.CONFIGS
    assert c["C1"].expert_bytes == 3 * 4096 * 14336 * 2
    assert round(c["C2"].expert_bytes / 1e6, 2) == 17.30
    assert round(c["C4"].expert_bytes / 1e6, 3) == 18.889
    assert c["C3"].cache_slots == 1536 and 5000 < c["C4"].cache_slots < 5200
    assert math.isclose(c["C3"].router_s, 0.714, abs_tol=1e-3)
