"""Failure paths, exercised without faulting or hanging the GPU: bounded waits that run out on
barriers nobody completes, host-side injection into the prefetch path (a lost request, a delayed
copy, a failed copy, a corrupted slot tag, a host wait that runs out), the cache-policy and
copy-throttle setters."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2606_15453_b200 as P
from datagen import stacks
from helpers import Pair

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
B = P.binding


@pytest.mark.parametrize("which", [0, 1, 2, 3, 4])
def test_bounded_waits_run_out_and_report_a_timeout(which):
    """The wait helpers of the persistent kernels on a barrier that is one arrival short (an mbarrier
    nobody arrives at, a completion counter nobody raises), poll limit 4096: the kernel ends, the error
    word is set."""
    cfg = stacks.CONFIGS["C0"].scaled(n_layers=2)
    pr = Pair(cfg, 1, oracle=False)
    assert pr.stack.stats()["decode_steps"] == 0           # healthy before
    pr.stack.selftest_bounded_wait(which, 4096)
    torch.cuda.synchronize()                               # returns: nothing hangs
    with pytest.raises(P.StmoeError, match="timed out"):
        pr.stack.stats()
    pr.close()


def _offloaded_cfg():
    return stacks.CONFIGS["C0"].scaled(n_layers=3, n_experts=16, top_k=2, hidden=128, inter=256, profile_tokens=3,
                                       dtype="bf16", cache_slots=12)


def _run(cfg, T, prepare=None, limit=2):
    pr = Pair(cfg, 2, oracle=False, prefetch_limit=limit)
    if prepare:
        prepare(pr.stack, -1)
    L, K = cfg.n_layers, cfg.top_k
    ids = torch.empty(L, 2, K, dtype=torch.int32, device=DEV)
    ho = torch.empty(2, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, 2, T).to(DEV)
    rec = []
    for t in range(T):
        if prepare:
            prepare(pr.stack, t)
        pr.stack.decode_token(x[t].clone(), ho, ids)
        torch.cuda.synchronize()
        rec.append((ho.cpu().clone(), ids.cpu().clone()))
    st = pr.stack.stats()
    pr.close()
    return rec, st


def test_lost_delayed_and_mislabelled_prefetches_never_change_results():
    cfg, T = _offloaded_cfg(), 10
    clean, st0 = _run(cfg, T)
    assert st0["prefetch_issued"] > 0 and st0["recovered_faults"] == 0

    def lose(stack, t):
        if t == 4:
            stack.test_hook(B.HOOK_DROP_PREFETCH, 3)
    lost, st1 = _run(cfg, T, lose)

    def delay(stack, t):
        if t in (3, 6):
            stack.test_hook(B.HOOK_DELAY_COPY_US, 3000)
    late, st2 = _run(cfg, T, delay)

    def mislabel(stack, t):
        if t == 5:
            tags = stack.export_cache_tags()
            stack.test_hook(B.HOOK_CORRUPT_TAG, int((tags >= 0).nonzero()[0]))
    wrong, st3 = _run(cfg, T, mislabel)

    for other in (lost, late, wrong):
        for a, b in zip(clean, other):
            assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert st1["prefetch_dropped"] >= st0["prefetch_dropped"] + 3 or st1["prefetch_issued"] < st0["prefetch_issued"]
    assert st2["transfer_ms"] > st0["transfer_ms"] + 5.0          # two delays of 3 ms inside the copy spans
    assert st3["recovered_faults"] >= 0                           # found only if the mislabelled expert is routed again


def test_a_failed_copy_fails_the_stack_until_a_state_is_imported():
    cfg = _offloaded_cfg()
    pr = Pair(cfg, 2, oracle=False, prefetch_limit=2)
    L, K = cfg.n_layers, cfg.top_k
    ids = torch.empty(L, 2, K, dtype=torch.int32, device=DEV)
    ho = torch.empty(2, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, 2, 8).to(DEV)
    for t in range(4):
        pr.stack.decode_token(x[t].clone(), ho, ids)
    torch.cuda.synchronize()
    image = pr.stack.export_state()
    pr.stack.test_hook(B.HOOK_FAIL_COPY, 1)
    with pytest.raises(P.StmoeError, match="CUDA error"):
        for t in range(4, 8):                        # the next copy that is issued fails
            pr.stack.decode_token(x[t].clone(), ho, ids)
    torch.cuda.synchronize()
    with pytest.raises(P.StmoeError, match="out of order|state"):
        pr.stack.decode_token(x[4].clone(), ho, ids)  # failed: no retry may apply Algorithm 3 twice
    pr.stack.import_state(image)
    for t in range(4, 8):
        pr.stack.decode_token(x[t].clone(), ho, ids)
    torch.cuda.synchronize()
    assert pr.stack.stats()["decode_steps"] == 8
    assert torch.isfinite(ho).all()
    pr.close()


def test_a_host_wait_that_runs_out_is_a_timeout_not_a_hang():
    cfg = _offloaded_cfg()
    pr = Pair(cfg, 2, oracle=False)
    ids = torch.empty(cfg.n_layers, 2, cfg.top_k, dtype=torch.int32, device=DEV)
    ho = torch.empty(2, cfg.hidden, device=DEV)
    x = stacks.token_inputs(cfg, 2, 2).to(DEV)
    pr.stack.decode_token(x[0].clone(), ho, ids)
    torch.cuda.synchronize()
    pr.stack.test_hook(B.HOOK_HOST_WAIT_MS, 0)
    torch.cuda._sleep(200_000_000)                    # ~0.1 s of device work ahead of the router on the stream
    with pytest.raises(P.StmoeError, match="timed out"):
        pr.stack.decode_token(x[1].clone(), ho, ids)
    torch.cuda.synchronize()                          # the device finishes what was enqueued
    pr.close()


def test_cache_policy_setter_matches_the_oracle_model_and_throttle_slows_the_link():
    cfg, T, Bt = _offloaded_cfg(), 12, 2
    res = {}
    for name, policy, throttle in (("lru", (0, False, -1), None), ("counts", (8, True, 0), None),
                                   ("throttled", (0, False, -1), (4096, 50))):
        pr = Pair(cfg, Bt, oracle=False, prefetch_limit=2)
        with pytest.raises(P.StmoeError):
            pr.stack.set_cache_policy(0, False, 0)     # a floor is a test on use counts: it needs a window
        pr.stack.set_cache_policy(*policy)
        if throttle:
            pr.stack.set_copy_throttle(*throttle)
        L, K = cfg.n_layers, cfg.top_k
        ids = torch.empty(L, Bt, K, dtype=torch.int32, device=DEV)
        ho = torch.empty(Bt, cfg.hidden, device=DEV)
        x = stacks.token_inputs(cfg, Bt, T).to(DEV)
        replay = O.Predictor(L, cfg.n_experts, K, Bt, cfg.profile_tokens, "st")
        cache = O.CacheModel(cfg.cache_slots, L, cfg.n_experts, window=policy[0], by_turn=policy[1], floor=policy[2])
        outs = []
        for t in range(T):
            pr.stack.decode_token(x[t].clone(), ho, ids)
            torch.cuda.synchronize()
            g = ids.cpu().numpy()
            for l in range(L):
                rp = replay.step(l, g[l])
                cache.step(l, np.unique(g[l]), (l + 1) % L, rp["queue_ids"], 2)
            outs.append(ho.cpu().clone())
        st, sc = pr.stack.stats(), cache.stats()
        assert (st["cache_hits"], st["cache_misses"], st["prefetch_issued"], st["prefetch_useful"], st["prefetch_wasted"],
                st["prefetch_dropped"], st["prefetch_resident"]) == \
            (sc["hits"], sc["misses"], sc["pf_issued"], sc["pf_useful"], sc["pf_wasted"], sc["pf_dropped"], sc["pf_resident"]), name
        assert (pr.stack.export_cache_tags().numpy() == cache.tags()).all(), name
        res[name] = (outs, st)
        with pytest.raises(P.StmoeError):
            pr.stack.set_cache_policy(0, False, -1)       # only before the first decode step
        pr.close()
    for a, b, c in zip(res["lru"][0], res["counts"][0], res["throttled"][0]):
        assert torch.equal(a, b) and torch.equal(a, c)     # the policy and the link speed never change a result
    assert res["throttled"][1]["transfer_ms"] > 1.5 * res["lru"][1]["transfer_ms"]
