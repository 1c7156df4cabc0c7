"""Edge cases of the CUDA path against the oracle: nothing left to decode,
ragged batches, odd lengths, no prompt, a window clipped at the sequence ends,
long sequences and many rows at the kernel level."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import dkv_oracle as O
from paper_2505_15781_b200 import binding as B
from paper_2505_15781_b200 import synth
from tests import gpu_util as U
from tests.test_gpu_ops import make_attention_case, oracle_attention

pytestmark = pytest.mark.gpu


def one_step(model, ms, x, m, pol, k=1, lo=None, hi=None, rows_bound=None, logits_rows=0, steps=1):
    b, L = x.shape
    cache = B.dkv_init_cache(model, b, L, 0, pol)
    tx, tm = torch.from_numpy(x).cuda(), torch.from_numpy(m).cuda()
    conf = torch.empty(b, L, device="cuda")
    pred = torch.empty(b, L, dtype=torch.int32, device="cuda")
    logits = torch.zeros(max(logits_rows, 1), ms.vocab, device="cuda") if logits_rows else None
    for _ in range(steps):
        B.dkv_step(cache, tx, tm, None, k, 0 if lo is None else lo, L if hi is None else hi,
                   int(m.sum(1).max()) if rows_bound is None else rows_bound, conf, pred, logits)
    return cache, conf.cpu().numpy(), pred.cpu().numpy(), None if logits is None else logits.cpu().numpy()


def test_nothing_masked_is_a_no_op_after_the_first_step():
    ms = synth.tiny_shape()
    _, model = U.build_pair(ms, 0, True)
    x = synth.make_prompt(2, 24, 1000, 0)
    m = np.zeros_like(x, dtype=np.uint8)
    cache, conf, pred, _ = one_step(model, ms, x, m, B.make_policy(B.DKV_POLICY_DECODE, 0), steps=3)
    assert np.isneginf(conf).all() and (pred == -1).all()
    assert B.dkv_status(cache) == 0
    st = B.dkv_get_stats(cache)
    assert st.steps == 3 and st.active_rows == 2 * 24          # the full first step, then no active row at all


def test_ragged_batch_odd_length_no_prompt():
    """Three sequences with 1, 9 and 20 masked positions, length 29, no prompt, fp32 check mode."""
    ms = synth.tiny_shape()
    W, model = U.build_pair(ms, 1, False)
    L = 29
    r = np.random.Generator(np.random.PCG64(5))
    x = r.integers(0, 1000, size=(3, L)).astype(np.int32)
    m = np.zeros((3, L), np.uint8)
    for b, n in enumerate((1, 9, 20)):
        pos = r.choice(L, size=n, replace=False)
        m[b, pos] = 1
        x[b, pos] = ms.mask_id
    n_head = int(m.sum())
    cache, conf, pred, logits = one_step(model, ms, x, m, B.make_policy(B.DKV_POLICY_DECODE, 0, max_head_rows=L),
                                         logits_rows=3 * L)
    assert B.dkv_status(cache) == 0
    off = 0
    for b in range(3):
        ref = O.vanilla_forward(U.oracle_model(ms), W, x[b].astype(np.int64))
        rows = np.nonzero(m[b])[0]
        assert np.abs(logits[off:off + len(rows)] - ref[rows]).max() < 1e-4
        for pos in rows:
            c, p = O.confidence(ref[pos], ms.mask_id)
            assert pred[b, pos] == p and abs(conf[b, pos] - c) < 2e-4 * c
        assert np.isneginf(conf[b][m[b] == 0]).all()
        off += len(rows)
    assert off == n_head


def test_more_tokens_requested_than_candidates_sets_the_status_bit():
    conf = torch.rand(2, 12, device="cuda")
    pred = torch.zeros(2, 12, dtype=torch.int32, device="cuda")
    tokens = torch.zeros(2, 12, dtype=torch.int32, device="cuda")
    masked = torch.zeros(2, 12, dtype=torch.uint8, device="cuda")
    masked[0, 5] = 1
    masked[1, 2:9] = 1
    chosen = torch.empty(2, 3, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.dkv_select_unmask(conf, pred, 2, 12, 0, 12, 3, tokens, masked, chosen, status)
    c = chosen.cpu().numpy()
    assert c[0].tolist() == [5, -1, -1] and (c[1] >= 2).all() and (c[1] < 9).all() and len(set(c[1])) == 3
    assert status.item() & 2


def test_greedy_window_clipped_at_both_ends():
    ms = synth.tiny_shape()
    W, model = U.build_pair(ms, 2, False)
    P, G = 0, 12
    pol = O.Policy(O.POLICY_GREEDY, 0, window=4)
    order = np.array([[0], [11], [1], [10], [5], [6], [2], [9], [3], [8], [4], [7]], dtype=np.int32)[:, None, :]
    prompts = np.zeros((1, 0), np.int32)
    tr = O.generate_one(U.oracle_model(ms), W, prompts[0], G, 1, pol, None, order[:, 0, :], keep_logits=True)
    run = U.ForcedRun(ms, model, 1, P, G, pol, 1)
    for st in tr:
        U.compare_step(run, [st], True, logit_tol_abs=1e-4)
        if st.t > 1:
            assert len(st.active) <= 6
    assert B.dkv_status(run.cache) == 0


@pytest.mark.parametrize("L,rows,hq,hkv", [(8192, 64, 4, 4), (4096, 300, 8, 1), (1000, 128, 14, 2)])
def test_attention_long_sequences_and_wide_groups(L, rows, hq, hkv):
    """Single-layer sweep sizes: up to 8192 slots, GQA groups of 7 and 8, a ragged last slot tile."""
    n_rows, tq, tk, tv, row_off = make_attention_case(9, 1, [rows], L, hq, hkv, 128, torch.float16)
    o = torch.zeros_like(tq)
    B.dkv_op_attention(tq, tk, tv, o, row_off, 1, rows, L, hq, hkv, 128, B.DKV_F16)
    ref, valid = oracle_attention(tq, tk, tv, n_rows, row_off.cpu().numpy())
    got = o.float().cpu().numpy()
    np.testing.assert_allclose(got[valid], ref[valid], atol=6 * 2.0 ** -11, rtol=6 * 2.0 ** -11)


def test_gemm_many_rows_and_all_four_projection_shapes():
    """Rows far beyond one tile (compute-bound regime) and the four LLaDA-shaped projections at 257 rows."""
    r = np.random.Generator(np.random.PCG64(11))
    for rows, n, k in [(2048, 512, 1024), (257, 12288, 4096), (257, 4096, 4096), (257, 4096, 12288)]:
        x = torch.from_numpy(r.standard_normal((rows, k)).astype(np.float32)).half().cuda()
        w = torch.from_numpy((r.standard_normal((n, k)) * 0.02).astype(np.float32)).half().cuda()
        out = torch.empty(rows, n, dtype=torch.float32, device="cuda")
        B.dkv_op_gemm(x, w, out, B.DKV_F16)
        ref = (x.double() @ w.double().T).cpu().numpy()          # library matmul in fp64 as the reference
        np.testing.assert_allclose(out.cpu().numpy(), ref, atol=3e-6 * k ** 0.5 * 4, rtol=1e-5)


@pytest.mark.parametrize("rows,L,hq,hkv", [(40, 700, 4, 4), (200, 1100, 8, 2)])
def test_attention_accumulator_rescale_path(rows, L, hq, hkv):
    """Scores whose maximum keeps growing along the slots (key norms rise 3x every 128 slots): the
    kernel has to move its reference exponent and rescale the output accumulator in almost every
    iteration, and, in between, works with probabilities above 1.  Both kernel shapes (the second case
    has more than 148 CTAs)."""
    n_rows, tq, tk, tv, row_off = make_attention_case(13, 1, [rows], L, hq, hkv, 128, torch.float16)
    q = torch.abs(tq.float())                       # positive queries: the score grows with the key norm
    grow = (3.0 ** (torch.arange(L, device="cuda") // 128).float()) * 0.02
    k = torch.abs(tk.float()) * grow[None, None, :, None]
    tq, tk = q.half(), k.half()
    o = torch.zeros_like(tq)
    B.dkv_op_attention(tq, tk, tv, o, row_off, 1, rows, L, hq, hkv, 128, B.DKV_F16)
    ref, valid = oracle_attention(tq, tk, tv, n_rows, row_off.cpu().numpy())
    np.testing.assert_allclose(o.float().cpu().numpy()[valid], ref[valid], atol=6 * 2.0 ** -11, rtol=6 * 2.0 ** -11)


HD128 = synth.ModelShape(2, 256, 2, 2, 128, 512, 1000, 999)     # head_dim 128: the tcgen05 attention kernel


@pytest.mark.parametrize("P,G", [(37, 40), (100, 92)])
def test_step_does_not_depend_on_what_the_arena_held(P, G):
    """Two layers, head_dim 128, a sequence length that is no multiple of the attention kernel's slot
    tile (64 or 128), the arena filled with 0xFF bytes (NaN patterns in fp16 and fp32) before the
    cache is initialised.  At step 1 layer 0 attends while layer 1's slots are still unwritten, and the
    last slot tile of layer 0's last head reaches past the sequence: nothing of that may leak into
    the result.  Compared with the oracle for a full step and two cached steps, on both head paths."""
    ms, pol = HD128, O.Policy(O.POLICY_DECODE, 0)
    W, model = U.build_pair(ms, 11, True)
    prompts = synth.make_prompt(2, P, ms.vocab - 1, 11)
    samplers = [O.Sampler(U.oracle_model(ms), W, prompts[b], G, 2, pol, None, None, "literal", keep_logits=True)
                for b in range(2)]
    run = U.ForcedRun(ms, model, 2, P, G, pol, 2, fused=True, arena_fill=0xFF)
    for _ in range(3):
        tr_t = [s.step() for s in samplers]
        err, sig, conf, pred = U.compare_step(run, tr_t, False, logit_tol_sigma=2e-2)
        assert np.isfinite(err)
    assert B.dkv_status(run.cache) == 0 and B.dkv_status(run.cache_f) == 0


def slot_tensors(cache, ms, layer, batch, L, dtype):
    """The K and V slots of one layer as torch views [batch, kv_heads, L, head_dim] into the arena."""
    kp, vp = B.dkv_cache_slots(cache, layer)
    n = batch * ms.n_kv_heads * L * ms.head_dim
    esz = torch.tensor([], dtype=dtype).element_size()
    out = []
    for ptr in (kp, vp):
        off = ptr - cache.arena.data_ptr()
        out.append(cache.arena[off:off + n * esz].view(dtype).view(batch, ms.n_kv_heads, L, ms.head_dim))
    return out


@pytest.mark.parametrize("bf16", [False, True])
def test_cache_slot_contents_match_the_oracles_cache(bf16):
    """Which step's K/V a position holds (Appendix A: a token's states enter the cache one step after it
    is decoded): after a full step and two cached steps every slot of every layer is compared with the
    oracle's position-addressed cache, stable rows (still holding an earlier step's K/V) and active rows
    alike.  fp32 mode: 1e-5 absolute; 16-bit mode: the operand and slot rounding of fp16 (2^-11 relative
    each, accumulated over the layers) -- 1e-2 of the tensor's rms."""
    ms = HD128 if bf16 else dataclasses.replace(synth.tiny_shape(), n_kv_heads=2)
    P, G, k, pol = 12, 20, 2, O.Policy(O.POLICY_DECODE, 0)
    W, model = U.build_pair(ms, 4, bf16)
    prompt = synth.make_prompt(1, P, ms.vocab - 1, 4)
    sampler = O.Sampler(U.oracle_model(ms), W, prompt[0], G, k, pol, None, None, "slots", keep_logits=True)
    run = U.ForcedRun(ms, model, 1, P, G, pol, k)
    L = P + G
    for _ in range(3):
        U.compare_step(run, [sampler.step()], False, logit_tol_abs=None if bf16 else 1e-4,
                       logit_tol_sigma=2e-2 if bf16 else None)
    assert (sampler.cache.written_step[:P] == 1).all()          # the prompt rows still hold step 1's K/V
    for layer in range(ms.n_layers):
        ks, vs = slot_tensors(run.cache, ms, layer, 1, L, torch.float16 if bf16 else torch.float32)
        for got, ref in ((ks, sampler.cache.K[layer]), (vs, sampler.cache.V[layer])):
            g = got[0].float().cpu().numpy().transpose(1, 0, 2)          # [L, kv_heads, head_dim] like the oracle
            tol = 1e-2 * np.sqrt(np.mean(ref * ref)) if bf16 else 1e-5
            assert np.abs(g - ref).max() <= tol, f"layer {layer}: slot contents differ by {np.abs(g - ref).max()}"


@pytest.mark.parametrize("ms", [synth.ModelShape(2, 328, 3, 3, 64, 344, 777, 776),      # nothing a multiple of 64
                                synth.ModelShape(1, 200, 2, 1, 128, 136, 515, 514)])
def test_widths_that_fill_neither_a_weight_block_nor_a_k_block(ms):
    """d_model, d_ffn and the projections' row counts are multiples of 8 only: the last 64-column block
    of every operand and the last 128-row block of every weight matrix are partly padding (zeros in the
    blocked fp16 copies, the copy engine's fill for the row operands), and the vocabulary ends inside a
    weight tile.  Full step, cached steps and a refresh against the oracle, both head paths."""
    from tests.test_gpu_step import run_forced
    worst = run_forced(ms, True, 2, 21, 12, 2, O.Policy(O.POLICY_DECODE, 3), 6, seed=13)
    assert worst < 2e-2
    worst = run_forced(ms, True, 3, 9, 8, 1, O.Policy(O.POLICY_PD, 0, isolated_prefill=True), None, seed=14)
    assert worst < 2e-2


def test_greedy_rejects_a_change_of_k_between_steps():
    """The window rule reads D_{t-1} with the k it was stored with."""
    ms = synth.tiny_shape()
    _, model = U.build_pair(ms, 0, False)
    cache = B.dkv_init_cache(model, 1, 16, 8, B.make_policy(B.DKV_POLICY_GREEDY, window=4, max_k=2))
    x = torch.zeros(1, 16, dtype=torch.int32, device="cuda")
    m = torch.zeros(1, 16, dtype=torch.uint8, device="cuda")
    m[0, 8:] = 1
    conf = torch.empty(1, 16, device="cuda")
    pred = torch.empty(1, 16, dtype=torch.int32, device="cuda")
    d = torch.tensor([[8, 9]], dtype=torch.int32, device="cuda")
    B.dkv_step(cache, x, m, d, 2, 8, 16, 8, conf, pred)
    with pytest.raises(B.DkvError) as e:
        B.dkv_step(cache, x, m, d, 1, 8, 16, 8, conf, pred)
    assert e.value.status == -2
    B.dkv_step(cache, x, m, d, 2, 8, 16, 8, conf, pred)
    assert B.dkv_status(cache) == 0


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """The bounded waits' error path, without a fault: the fused tails of one handle are told to expect an
    arrival that never comes and to give up after 2 million clocks (about a millisecond).  The step must
    come back, dkv_status must show the wait bit (8), and a fresh handle on the same device must then
    reproduce the oracle."""
    ms, P, G, pol = HD128, 20, 12, O.Policy(O.POLICY_DECODE, 0)
    W, model = U.build_pair(ms, 6, True)
    x, m = synth.initial_state(synth.make_prompt(1, P, ms.vocab - 1, 6), G, ms.mask_id)
    tx, tm = torch.from_numpy(x).cuda(), torch.from_numpy(m).cuda()
    conf = torch.empty(1, P + G, device="cuda")
    pred = torch.empty(1, P + G, dtype=torch.int32, device="cuda")
    cache = B.dkv_init_cache(model, 1, P + G, P, U.gpu_policy(pol))
    B.dkv_debug_tail_wait(cache, 2_000_000, True)
    B.dkv_step(cache, tx, tm, None, 1, P, P + G, G, conf, pred)
    torch.cuda.synchronize()
    assert B.dkv_status(cache) & 8
    del cache
    prompt = synth.make_prompt(1, P, ms.vocab - 1, 6)
    sampler = O.Sampler(U.oracle_model(ms), W, prompt[0], G, 1, pol, None, None, "literal", keep_logits=True)
    run = U.ForcedRun(ms, model, 1, P, G, pol, 1, fused=True)
    for _ in range(2):
        U.compare_step(run, [sampler.step()], False, logit_tol_sigma=2e-2)
    assert B.dkv_status(run.cache) == 0 and B.dkv_status(run.cache_f) == 0
