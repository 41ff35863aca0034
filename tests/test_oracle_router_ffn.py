"""Pins for the oracle's floating-point parts: storage decoders, RMSNorm, gating
logits, softmax, top-K selection, SwiGLU expert FFN and the weighted expert sum."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle as O
from datagen import rng


def _randn(n, tag):
    return rng.normal(n, rng.stream_key(99, tag)).numpy()


def test_bf16_decoder_matches_torch_on_every_code():
    codes = torch.arange(65536, dtype=torch.int32).to(torch.uint16)
    want = codes.view(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([O.lib().orc_bf16_to_f32(int(c)) for c in range(65536)], dtype=np.float32)
    ok = (got == want) | (np.isnan(got) & np.isnan(want))
    assert ok.all()


def test_e4m3_decoder_matches_torch_on_every_code():
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    want = codes.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = np.array([O.lib().orc_e4m3_to_f32(int(c)) for c in range(256)], dtype=np.float32)
    ok = (got == want) | (np.isnan(got) & np.isnan(want))
    assert ok.all()
    assert got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9


def test_rmsnorm_matches_library_routine():
    h = _randn(384, 1) * 3.0
    want = F.rms_norm(torch.from_numpy(h).double(), (384,), eps=1e-6).numpy()
    got = O.rmsnorm(h, 1e-6)
    assert np.abs(got - want).max() < 1e-6
    assert abs(np.sqrt(np.mean(got.astype(np.float64) ** 2)) - 1.0) < 1e-5


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_router_logits_match_matmul(dtype):
    E, H = 12, 200   # non-square: a transposed operand cannot pass
    W = torch.from_numpy(_randn(E * H, 2).reshape(E, H))
    if dtype == "bf16":
        W = W.to(torch.bfloat16)
    x = _randn(H, 3)
    want = (W.double() @ torch.from_numpy(x).double()).numpy()
    got = O.router_logits(x, W.contiguous(), dtype)
    assert np.abs(got - want).max() < 1e-5


def test_softmax_matches_library_and_sums_to_one():
    z = _randn(64, 4) * 5
    want = torch.softmax(torch.from_numpy(z).double(), 0).numpy()
    got = O.softmax(z)
    assert np.abs(got - want).max() < 1e-7
    assert abs(got.astype(np.float64).sum() - 1.0) < 1e-6
    big = O.softmax(np.array([1000.0, 1000.0, -1000.0], dtype=np.float32))
    assert np.allclose(big, [0.5, 0.5, 0.0])


@pytest.mark.parametrize("E,K", [(8, 2), (9, 3), (64, 6), (128, 8), (5, 5), (7, 1)])
def test_topk_equals_full_sort(E, K):
    for trial in range(20):
        z = _randn(E, 100 + trial)
        if trial % 3 == 0:                       # force exact ties, also across the K-th place
            z = np.round(z * 2) / 2
        order = sorted(range(E), key=lambda j: (-z[j], j))   # value desc, lower id first
        want = sorted(order[:K])
        ids, gap = O.topk(z, K)
        assert ids.tolist() == want
        if K < E:
            assert gap == pytest.approx(z[order[K - 1]] - z[order[K]])
        else:
            assert gap == np.inf


def test_route_weights_are_unrenormalised_probabilities():
    E, H, K = 8, 64, 2
    W = torch.from_numpy(_randn(E * H, 5).reshape(E, H)).contiguous()
    h = _randn(H, 6) * 2
    r = O.route(h, W, "f32", K)
    x = F.rms_norm(torch.from_numpy(h).double(), (H,), eps=1e-6)
    s = torch.softmax(W.double() @ x, 0)
    top = torch.topk(s, K).indices.sort().values
    assert r["ids"].tolist() == top.tolist()
    assert np.abs(r["w"] - s[top].numpy()).max() < 1e-6
    assert r["w"].sum() < 1.0
    rn = O.route(h, W, "f32", K, renorm=True)
    assert abs(rn["w"].sum() - 1.0) < 1e-6
    # a planted exact tie at the K-th place is flagged
    order = torch.topk(s, K + 1).indices.tolist()
    kth, nxt = order[K - 1], order[K]
    W2 = W.clone()
    W2[nxt] = W2[kth]
    r2 = O.route(h, W2, "f32", K)
    assert r2["near_tie"] == 1 and r["near_tie"] == 0
    assert min(kth, nxt) in r2["ids"] and max(kth, nxt) not in r2["ids"]   # tie -> lower id


def _weights(H, I, dtype, tag):
    w = {}
    for i, (name, shape) in enumerate((("gate", (I, H)), ("up", (I, H)), ("down", (H, I)))):
        m = torch.from_numpy(_randn(shape[0] * shape[1], tag * 10 + i).reshape(shape)) * 0.1
        if dtype == "bf16":
            m = m.to(torch.bfloat16)
        if dtype == "fp8":
            amax = m.abs().amax(1)
            sc = (amax / 448).to(torch.bfloat16)
            w[name + "_scale"] = sc.contiguous()
            m = (m / sc.float()[:, None]).clamp(-448, 448).to(torch.float8_e4m3fn)
        w[name] = m.contiguous()
    return w


def _dequant(w, name):
    m = w[name].to(torch.float32)
    if name + "_scale" in w:
        m = m * w[name + "_scale"].to(torch.float32)[:, None]
    return m.double()


@pytest.mark.parametrize("dtype", ["f32", "bf16", "fp8"])
def test_expert_ffn_matches_library_ops(dtype):
    H, I = 48, 80
    w = _weights(H, I, dtype, 7)
    x = _randn(H, 8)
    xd = torch.from_numpy(x).double()
    want = (_dequant(w, "down") @ (F.silu(_dequant(w, "gate") @ xd) * (_dequant(w, "up") @ xd)))
    got = O.expert_ffn(x, w, dtype)
    assert np.abs(got - want.numpy()).max() < 1e-5 * max(1.0, float(want.abs().max()))


def test_expert_ffn_brute_force_loop():
    H, I = 5, 7
    w = _weights(H, I, "f32", 9)
    x = _randn(H, 10)
    g, u, d = (w[k].double().tolist() for k in ("gate", "up", "down"))
    a = []
    for i in range(I):
        gi = sum(g[i][j] * float(x[j]) for j in range(H))
        ui = sum(u[i][j] * float(x[j]) for j in range(H))
        a.append(gi / (1.0 + np.exp(-gi)) * ui)
    want = [sum(d[h][i] * a[i] for i in range(I)) for h in range(H)]
    assert np.abs(O.expert_ffn(x, w, "f32") - np.array(want)).max() < 1e-6


def test_combine_linearity_and_zero_weights():
    H, K = 32, 3
    h = _randn(H, 11)
    yk = _randn(K * H, 12).reshape(K, H)
    ys = _randn(2 * H, 13).reshape(2, H)
    w = np.array([0.5, 0.25, 0.125], dtype=np.float32)
    out = O.combine(h, ys, yk, w, 0.1)
    want = h + 0.1 * (ys.sum(0) + (w[:, None] * yk).sum(0))
    assert np.abs(out - want).max() < 1e-6
    out2 = O.combine(h, None, yk, 2 * w, 0.1)
    out1 = O.combine(h, None, yk, w, 0.1)
    assert np.abs((out2 - h) - 2 * (out1 - h)).max() < 1e-6
    assert (O.combine(h, None, np.zeros((K, H), np.float32), w, 0.1) == h).all()
