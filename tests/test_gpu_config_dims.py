"""Parity at the benchmark configurations' own matrix sizes, on short stacks so the CPU oracle
stays affordable: the fp8 tensor-core kernels at the Qwen3-235B shape (hidden 4096,
intermediate 1536: sixteen K stages per gate/up task and the down-split geometry of that
shape), the persistent bf16 tensor-core kernel at the Mixtral shape (hidden 4096, intermediate
14336), and the slot manager at the Qwen3-30B configuration's full depth and slot count."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2606_15453_b200 as P
from datagen import stacks
from helpers import Pair, cache_policy, check_layer, decode_tokens_vs_oracle as _decode_token_vs_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_fp8_tensor_core_kernels_at_c4_matrix_sizes_batch32():
    """Per-layer dense_group_kernel launches with fp8 operands at hidden 4096 / intermediate 1536,
    teacher-forced layer by layer."""
    cfg = stacks.CONFIGS["C4"].scaled(n_layers=2, n_experts=32, profile_tokens=1, cache_slots=0)
    assert (cfg.hidden, cfg.inter, cfg.dtype) == (4096, 1536, "fp8")
    B = 32
    pr = Pair(cfg, B)
    x = stacks.token_inputs(cfg, B, 2).numpy()
    skipped = 0
    for t in range(2):
        h = x[t]
        for l in range(cfg.n_layers):
            o = pr.oracle.layer_step(l, h)
            g = pr.gpu_step(l, h)
            skipped += check_layer(cfg, g, o, h, where=f"t={t} l={l}")
            h = o["h_out"]
    st = pr.stack.stats()
    assert st["kernel_launches"] == 2 * cfg.n_layers * 6 + 1     # router, predictor, cast, gate/up, down, sum
    assert skipped <= B // 2
    pr.close()


@pytest.mark.parametrize("B,T", [(4, 3), (32, 2)])
def test_fp8_persistent_tensor_core_kernel_at_c4_matrix_sizes(B, T):
    cfg = stacks.CONFIGS["C4"].scaled(n_layers=2, n_experts=32, profile_tokens=1, cache_slots=0)
    st = _decode_token_vs_oracle(cfg, B, T, min_checked=(T - 1) * B)
    assert st["kernel_launches"] <= T + 1        # one persistent launch per step (+ the table build)


def test_bf16_persistent_tensor_core_kernel_at_c1_matrix_sizes_batch4():
    free = torch.cuda.mem_get_info()[0]
    cfg = stacks.CONFIGS["C1"].scaled(n_layers=2, profile_tokens=1)
    assert (cfg.hidden, cfg.inter, cfg.dtype) == (4096, 14336, "bf16")
    if free < 2 * cfg.n_experts * cfg.expert_bytes + (8 << 30):
        pytest.skip("not enough free HBM")
    st = _decode_token_vs_oracle(cfg, 4, 3, min_checked=6)
    assert st["kernel_launches"] <= 3 + 1


@pytest.mark.parametrize("B", [1, 16])
def test_slot_manager_at_c3_depth_and_slot_count(B):
    """The Qwen3-30B configuration's 48 layers, 128 experts, top-8 and 1536 slots with small
    matrices: 40 decode steps, every counter and every slot tag integer-exact against the
    oracle's cache model driven by the GPU's routing and the replayed prefetch queue."""
    cfg = stacks.CONFIGS["C3"].scaled(hidden=64, inter=64, profile_tokens=4)
    assert (cfg.n_layers, cfg.n_experts, cfg.top_k, cfg.cache_slots) == (48, 128, 8, 1536)
    limit = 4 if B > 1 else 0
    pr = Pair(cfg, B, prefetch_limit=limit, oracle=False)
    L, K, T = cfg.n_layers, cfg.top_k, 40
    x = stacks.token_inputs(cfg, B, T).to(DEV)
    ids = torch.empty(L, B, K, dtype=torch.int32, device=DEV)
    pred = torch.empty(L, B, pr.stack.max_pred, dtype=torch.int32, device=DEV)
    npred = torch.empty(L, B, dtype=torch.int32, device=DEV)
    ho = torch.empty(B, cfg.hidden, device=DEV)
    replay = O.Predictor(L, cfg.n_experts, K, B, cfg.profile_tokens, "st")
    policy = cache_policy(cfg, B)
    assert policy["by_turn"] == (B == 16)       # batch 16 touches 48 x 128 keys per step, more than 1536 slots
    cache = O.CacheModel(cfg.cache_slots, L, cfg.n_experts, **policy)
    for t in range(T):
        pr.stack.decode_token(x[t], ho, ids, None, pred, npred)
        torch.cuda.synchronize()
        g_ids, g_pred, g_np = ids.cpu().numpy(), pred.cpu().numpy(), npred.cpu().numpy()
        for l in range(L):
            rp = replay.step(l, g_ids[l])
            assert g_np[l].tolist() == rp["n_pred"].tolist() and (g_pred[l] == rp["pred_ids"]).all(), (t, l)
            cache.step(l, np.unique(g_ids[l]), (l + 1) % L, rp["queue_ids"], limit)
    st, sc = pr.stack.stats(), cache.stats()
    assert (st["cache_hits"], st["cache_misses"], st["prefetch_issued"], st["prefetch_useful"],
            st["prefetch_wasted"], st["prefetch_dropped"], st["prefetch_resident"]) == \
        (sc["hits"], sc["misses"], sc["pf_issued"], sc["pf_useful"], sc["pf_wasted"],
         sc["pf_dropped"], sc["pf_resident"])
    assert (pr.stack.export_cache_tags().numpy() == cache.tags()).all()
    assert st["cache_hits"] + st["cache_misses"] > 0 and st["prefetch_issued"] > 0
    assert pr.stack.export_state() == replay.export()
    pr.close()
