"""Full-size parity: the benchmark workload (Mixtral-shaped bf16 stack, 32 layers, 90 GB of
resident experts, batch 1) through the same entry point and launch configuration bench.py
times (stmoe_decode_token -> persistent decode-step kernel), against the CPU oracle running
its own residual stream for whole decode steps; and the DeepSeek-V2-Lite-shaped stack at batch 8
through the persistent tensor-core kernel."""
import numpy as np
import pytest
import torch

import oracle as O
from datagen import stacks
from helpers import TOL, Pair, decode_tokens_vs_oracle, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_c1_full_size_decode_steps_match_oracle():
    free = torch.cuda.mem_get_info()[0]
    cfg = stacks.CONFIGS["C1"].scaled(profile_tokens=1)
    need = cfg.n_layers * cfg.n_experts * cfg.expert_bytes + (8 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free HBM, {free >> 30} GiB available")
    T = 3
    pr = Pair(cfg, 1)
    L, K = cfg.n_layers, cfg.top_k
    x = stacks.token_inputs(cfg, 1, T)
    ids = torch.empty(L, 1, K, dtype=torch.int32, device=DEV)
    w = torch.empty(L, 1, K, dtype=torch.float32, device=DEV)
    pred = torch.empty(L, 1, pr.stack.max_pred, dtype=torch.int32, device=DEV)
    npred = torch.empty(L, 1, dtype=torch.int32, device=DEV)
    flags = torch.empty(L, 1, dtype=torch.int32, device=DEV)
    ho = torch.empty(1, cfg.hidden, device=DEV)
    replay = O.Predictor(L, cfg.n_experts, K, 1, cfg.profile_tokens, "st")
    checked_outputs = 0
    for t in range(T):
        pr.stack.decode_token(x[t].to(DEV), ho, ids, w, pred, npred, flags)
        torch.cuda.synchronize()
        g_ids, g_pred, g_np = ids.cpu().numpy(), pred.cpu().numpy(), npred.cpu().numpy()
        # the predictor is bit-exact on the GPU's own routing, always
        for l in range(L):
            rp = replay.step(l, g_ids[l])
            assert g_np[l].tolist() == rp["n_pred"].tolist() and (g_pred[l] == rp["pred_ids"]).all(), (t, l)
        h_ref, per = pr.oracle.decode_token(x[t].numpy())     # about 15 s of CPU per step
        o_ids = np.stack([r["ids"] for r in per])
        ties = sum(int(r["ties"].sum()) for r in per) + int(flags.sum())
        if (o_ids != g_ids).any():
            assert ties > 0, "routing diverged from the oracle without a near tie"
        else:
            assert np.abs(w.cpu().numpy() - np.stack([r["w"] for r in per])).max() < 2e-5
            assert rel_err(ho.cpu().numpy(), h_ref) <= TOL["bf16"]
            assert rel_err(ho.cpu().numpy() - x[t].numpy(), h_ref - x[t].numpy()) <= 5e-3
            checked_outputs += 1
    assert pr.stack.export_state() == replay.export()
    assert checked_outputs >= T - 1
    pr.close()


def test_c2_full_size_batch8_tensor_core_step_matches_oracle():
    """C2 at full size (26 layers, 64 + 2 experts, 29.7 GB) with eight sequences: the launch
    bench.py times for `--workload C2 --batch 8` (decode_token_dense_kernel)."""
    free = torch.cuda.mem_get_info()[0]
    cfg = stacks.CONFIGS["C2"].scaled(profile_tokens=1)
    need = cfg.n_layers * (cfg.n_experts + cfg.n_shared) * cfg.expert_bytes + (8 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free HBM, {free >> 30} GiB available")
    B, T = 8, 3
    pr = Pair(cfg, B)
    L, K = cfg.n_layers, cfg.top_k
    x = stacks.token_inputs(cfg, B, T)
    ids = torch.empty(L, B, K, dtype=torch.int32, device=DEV)
    w = torch.empty(L, B, K, dtype=torch.float32, device=DEV)
    pred = torch.empty(L, B, pr.stack.max_pred, dtype=torch.int32, device=DEV)
    npred = torch.empty(L, B, dtype=torch.int32, device=DEV)
    flags = torch.empty(L, B, dtype=torch.int32, device=DEV)
    ho = torch.empty(B, cfg.hidden, device=DEV)
    replay = O.Predictor(L, cfg.n_experts, K, B, cfg.profile_tokens, "st")
    checked = 0
    for t in range(T):
        pr.stack.decode_token(x[t].to(DEV), ho, ids, w, pred, npred, flags)
        torch.cuda.synchronize()
        g_ids, g_pred, g_np = ids.cpu().numpy(), pred.cpu().numpy(), npred.cpu().numpy()
        for l in range(L):   # the predictor is bit-exact on the GPU's own routing, always
            rp = replay.step(l, g_ids[l])
            assert g_np[l].tolist() == rp["n_pred"].tolist() and (g_pred[l] == rp["pred_ids"]).all(), (t, l)
        # every step (about 10 s of CPU each), layer by layer so that the oracle's input of every
        # layer is at hand
        h_l, hs, per = x[t].numpy(), [], []
        for l in range(L):
            hs.append(h_l)
            per.append(pr.oracle.layer_step(l, h_l))
            h_l = per[-1]["h_out"]
        h_ref = h_l
        o_ids = np.stack([r["ids"] for r in per])
        got = ho.cpu().numpy()
        for b in range(B):
            # a sequence is comparable while its routing agrees with the oracle's in every layer
            if (o_ids[:, b] != g_ids[:, b]).any():
                if sum(int(r["ties"][b]) for r in per) + int(flags[:, b].sum()) > 0:
                    continue
                # Free-running streams: the tensor-core path rounds its operands to bf16, so after a few
                # layers its hidden state differs from the oracle's at the 1e-3 level and a routing
                # decision may part where the oracle's logit gap is of that order (the strict check,
                # same input per layer, is test_config_shapes_teacher_forced).  Anything wider is a bug.
                l0 = int(np.flatnonzero((o_ids[:, b] != g_ids[:, b]).any(axis=1))[0])
                z = np.sort(O.route(hs[l0][b], pr.oracle.router_w[l0], cfg.router_dtype, K, cfg.rms_eps)["z"])[::-1]
                assert z[K - 1] - z[K] < 1e-2, f"sequence {b} layer {l0}: routing parted at a logit gap of {z[K - 1] - z[K]}"
                continue
            assert rel_err(got[b], h_ref[b]) <= TOL["bf16"], b
            assert rel_err(got[b] - x[t][b].numpy(), h_ref[b] - x[t][b].numpy()) <= 2e-2, b
            checked += 1
    assert pr.stack.export_state() == replay.export()
    assert checked >= T * B // 2
    st = pr.stack.stats()
    assert st["kernel_launches"] <= T + 1      # one persistent launch per step (+ the table build)
    pr.close()


def test_c2_full_size_batch1_single_sequence_kernel_matches_oracle():
    """C2 at full size with one sequence: the launch bench.py times for `--workload C2`
    (decode_token_fused_kernel, 26 layers, shared experts), every decode step against the oracle."""
    free = torch.cuda.mem_get_info()[0]
    cfg = stacks.CONFIGS["C2"].scaled(profile_tokens=1)
    need = cfg.n_layers * (cfg.n_experts + cfg.n_shared) * cfg.expert_bytes * 4 // 3 + (8 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free HBM, {free >> 30} GiB available")
    st = decode_tokens_vs_oracle(cfg, 1, 4, min_checked=3)
    assert st["kernel_launches"] <= 4 + 1          # one launch per decode step (+ the table build)
