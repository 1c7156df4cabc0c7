"""Checkpoint / resume of a generation: the state a handle carries between two steps (cached K/V,
the stored M_{t-1} / D_{t-1}, counters, provenance) exported to host memory and imported into a fresh
handle.  The resumed handle must go on matching the ORACLE step by step, across refresh steps, and be
bit-identical to the handle that was never interrupted."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import dkv_oracle as O
from paper_2505_15781_b200 import binding as B
from paper_2505_15781_b200 import synth
from tests import gpu_util as U
from tests.test_gpu_edges import slot_tensors
from tests.test_gpu_step import oracle_traces

pytestmark = pytest.mark.gpu

GQA = dataclasses.replace(synth.tiny_shape(), n_kv_heads=2)


def move_state(src, dst):
    blob = torch.empty(B.dkv_cache_state_bytes(src) + 64, dtype=torch.uint8)
    B.dkv_cache_export(src, blob)
    B.dkv_cache_import(dst, blob)
    return blob


def slots_of(cache, ms, batch, L, dtype):
    return [t for layer in range(ms.n_layers) for t in slot_tensors(cache, ms, layer, batch, L, dtype)]


def destroy(cache):
    assert B.load().dkv_cache_destroy(cache.handle) == 0
    cache.handle = None


@pytest.mark.parametrize("pol,k,block,order,cut", [
    (O.Policy(O.POLICY_DECODE, 4), 2, 8, False, 3),                 # resume inside an interval, one step before a refresh
    (O.Policy(O.POLICY_DECODE, 4), 1, None, False, 4),              # resume right after a refresh step
    (O.Policy(O.POLICY_PD, 3, isolated_prefill=True), 2, None, False, 1),
    (O.Policy(O.POLICY_PREFILL, shift=2), 1, None, False, 5),
    (O.Policy(O.POLICY_GREEDY, 4, window=4), 1, None, True, 6),     # D_{t-1} travels with the state
    (O.Policy(O.POLICY_GREEDY, 0, window=2, window_center=O.CENTER_CUR), 2, None, True, 2),
    (O.Policy(O.POLICY_DECODE, 0, delay=0), 1, None, False, 7),
])
@pytest.mark.parametrize("bf16", [False, True])
def test_resumed_handle_matches_the_oracle_and_the_uninterrupted_handle(pol, k, block, order, cut, bf16):
    ms, batch, P, G, seed = GQA, 2, 11, 16, 5
    W, model = U.build_pair(ms, seed, bf16)
    ordr = synth.random_order(batch, P, G, k, seed) if order else None
    traces = oracle_traces(ms, W, batch, P, G, k, pol, block, seed, ordr)
    greedy = pol.kind == O.POLICY_GREEDY
    tol = dict(logit_tol_abs=None, logit_tol_sigma=2e-2) if bf16 else dict(logit_tol_abs=1e-4, logit_tol_sigma=None)
    whole = U.ForcedRun(ms, model, batch, P, G, pol, k, fused=bf16)             # never interrupted
    first = U.ForcedRun(ms, model, batch, P, G, pol, k, fused=bf16)
    for t in range(cut):
        tr_t = [tr[t] for tr in traces]
        U.compare_step(whole, tr_t, greedy, **tol)
        U.compare_step(first, tr_t, greedy, **tol)
    # a fresh pair of handles in arenas full of 0xFF bytes takes over from `first`
    second = U.ForcedRun(ms, model, batch, P, G, pol, k, fused=bf16, arena_fill=0xFF)
    move_state(first.cache, second.cache)
    if bf16:
        move_state(first.cache_f, second.cache_f)
    destroy(first.cache)
    if bf16:
        destroy(first.cache_f)
    for t in range(cut, len(traces[0])):
        tr_t = [tr[t] for tr in traces]
        U.compare_step(whole, tr_t, greedy, **tol)
        U.compare_step(second, tr_t, greedy, **tol)
        n_head = sum(len(s.head_rows) for s in tr_t)         # rows past these hold earlier steps' logits
        assert torch.equal(whole.logits[:n_head], second.logits[:n_head]), f"step {t + 1}: not the uninterrupted run's logits"
        assert torch.equal(whole.conf, second.conf) and torch.equal(whole.pred, second.pred)
        assert torch.equal(whole.prov, second.prov) and torch.equal(whole.inv, second.inv)
        if bf16:
            assert torch.equal(whole.conf_f, second.conf_f) and torch.equal(whole.pred_f, second.pred_f)
    dt = torch.float16 if bf16 else torch.float32
    for a, b in zip(slots_of(whole.cache, ms, batch, P + G, dt), slots_of(second.cache, ms, batch, P + G, dt)):
        assert torch.equal(a, b)
    sa, sb = B.dkv_get_stats(whole.cache), B.dkv_get_stats(second.cache)
    assert (sa.steps, sa.refresh_steps, sa.active_rows, sa.total_rows) == (sb.steps, sb.refresh_steps, sb.active_rows,
                                                                          sb.total_rows)
    assert sa.cache_ratio == sb.cache_ratio
    assert abs(sb.cache_ratio - np.mean([O.cache_ratio(tr) for tr in traces])) < 1e-12
    assert B.dkv_status(second.cache) == 0


def test_free_running_generation_resumed_in_the_middle_ends_in_the_same_tokens():
    """dkv_generate for the first half, export, import into a new handle, dkv_generate for the rest:
    the tokens, the decoding order and the provenance equal those of one uninterrupted call."""
    ms, batch, P, G, k, seed = GQA, 3, 9, 24, 2, 11
    pol = O.Policy(O.POLICY_DECODE, 4)
    W, model = U.build_pair(ms, seed, True)
    T = G // k
    prompts = synth.make_prompt(batch, P, 1000, seed)

    def fresh():
        x = torch.full((batch, P + G), ms.mask_id, dtype=torch.int32, device="cuda")
        x[:, :P] = torch.tensor(prompts, dtype=torch.int32)
        m = torch.zeros(batch, P + G, dtype=torch.uint8, device="cuda")
        m[:, P:] = 1
        return x, m, torch.full((T, batch, k), -7, dtype=torch.int32, device="cuda")
    x0, m0, ch0 = fresh()
    c0 = B.dkv_init_cache(model, batch, P + G, P, U.gpu_policy(pol, max_k=k))
    B.dkv_generate(c0, x0, m0, None, k, 8, 0, ch0)
    x1, m1, ch1 = fresh()
    c1 = B.dkv_init_cache(model, batch, P + G, P, U.gpu_policy(pol, max_k=k))
    B.dkv_generate(c1, x1, m1, None, k, 8, 5, ch1)
    c2 = B.dkv_init_cache(model, batch, P + G, P, U.gpu_policy(pol, max_k=k))
    move_state(c1, c2)
    destroy(c1)
    B.dkv_generate(c2, x1, m1, None, k, 8, 0, ch1)          # continues at step 6
    torch.cuda.synchronize()
    assert int(m1.sum()) == 0
    assert torch.equal(x0, x1) and torch.equal(ch0, ch1)
    p0, p1 = torch.empty_like(x0), torch.empty_like(x0)
    B.dkv_get_provenance(c0, p0)
    B.dkv_get_provenance(c2, p1)
    torch.cuda.synchronize()
    assert torch.equal(p0, p1)
    assert B.dkv_get_stats(c0).active_rows == B.dkv_get_stats(c2).active_rows


def test_import_refuses_what_does_not_fit_the_handle():
    ms, seed = GQA, 2
    W, model = U.build_pair(ms, seed, False)
    pol = U.gpu_policy(O.Policy(O.POLICY_DECODE, 4), max_k=1)
    a = B.dkv_init_cache(model, 1, 24, 8, pol)
    need = B.dkv_cache_state_bytes(a)
    blob = torch.zeros(need, dtype=torch.uint8)
    lib = B.load()

    def rc_export(c, t, n):
        return lib.dkv_cache_export(c.handle, t.data_ptr(), n, None)

    def rc_import(c, t, n):
        return lib.dkv_cache_import(c.handle, t.data_ptr(), n, None)
    assert rc_export(a, blob, need - 1) == -4                       # too small
    assert rc_import(a, blob, need) == -1                           # zeros: not an exported state
    assert rc_export(a, blob, need) == 0
    assert rc_import(a, blob, need) == 0                            # its own state
    assert rc_import(a, blob, need - 1) == -2                       # truncated
    for other in (B.dkv_init_cache(model, 1, 32, 8, pol),           # another length
                  B.dkv_init_cache(model, 2, 24, 8, pol),           # another batch
                  B.dkv_init_cache(model, 1, 24, 9, pol),           # another prompt length
                  B.dkv_init_cache(model, 1, 24, 8, U.gpu_policy(O.Policy(O.POLICY_DECODE, 5), max_k=1)),
                  B.dkv_init_cache(model, 1, 24, 8, U.gpu_policy(O.Policy(O.POLICY_PD, 4), max_k=1))):
        big = torch.zeros(max(need, B.dkv_cache_state_bytes(other)), dtype=torch.uint8)
        big[:need] = blob
        assert rc_import(other, big, big.numel()) == -2
    bad = blob.clone()
    bad[8] = 99                                                     # version field
    assert rc_import(a, bad, need) == -1
    assert B.dkv_status(a) == 0
