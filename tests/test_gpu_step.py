"""Step-level parity of the CUDA path against the oracle on the same seeded
inputs, through the C ABI.  Forced-trajectory mode: the library is fed the
oracle's (x_t, M_t) each step; index maps, provenance and selection must be
bit-exact, logits within 1e-4 (fp32 check mode) or 2e-2 * sigma(logits) (bf16)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import dkv_oracle as O
from paper_2505_15781_b200 import binding as B
from paper_2505_15781_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu

F32_TOL = 1e-4
BF16_TOL_SIGMA = 2e-2


def oracle_traces(ms, W, batch, P, G, k, pol, block=None, seed=0, order=None):
    prompts = synth.make_prompt(batch, P, min(1000, ms.vocab - 1), seed)
    out = []
    for b in range(batch):
        ordb = order[:, b, :] if order is not None else None
        out.append(O.generate_one(U.oracle_model(ms), W, prompts[b], G, k, pol, block, ordb, form="literal",
                                  keep_logits=True))
    return out


def run_forced(ms, bf16, batch, P, G, k, pol, block=None, seed=0, with_order=False, act=None, tol_sigma=BF16_TOL_SIGMA):
    W, model = U.build_pair(ms, seed, bf16, act=act)
    order = synth.random_order(batch, P, G, k, seed) if with_order else None
    traces = oracle_traces(ms, W, batch, P, G, k, pol, block, seed, order)
    run = U.ForcedRun(ms, model, batch, P, G, pol, k, fused=bf16)     # 16-bit: both head paths, every step
    greedy = pol.kind == O.POLICY_GREEDY
    worst = 0.0
    for t in range(len(traces[0])):
        tr_t = [tr[t] for tr in traces]
        err, sig, conf, pred = U.compare_step(run, tr_t, greedy,
                                              logit_tol_abs=None if bf16 else F32_TOL,
                                              logit_tol_sigma=tol_sigma if bf16 else None)
        worst = max(worst, err / sig)
        for b, s in enumerate(tr_t):
            hr = s.head_rows
            if not bf16:
                np.testing.assert_array_equal(pred[b][hr], s.pred[hr])
                np.testing.assert_allclose(conf[b][hr], s.conf[hr], rtol=2e-4, atol=1e-7)
    assert B.dkv_status(run.cache) == 0
    st = B.dkv_get_stats(run.cache)
    assert st.steps == len(traces[0])
    assert abs(st.cache_ratio - np.mean([O.cache_ratio(tr) for tr in traces])) < 1e-12
    return worst


def test_config1_fp32_decode_every_step():
    """Tiny model, prompt 32 + 32 masked, 32 steps, Decode, refresh every 8."""
    run_forced(synth.tiny_shape(), False, 1, 32, 32, 1, O.Policy(O.POLICY_DECODE, 8))


def test_config1_bf16_weights_decode_every_step():
    """bf16 weights, fp16 activations and cache (the benchmark's mode): 2e-2 sigma."""
    worst = run_forced(synth.tiny_shape(), True, 1, 32, 32, 1, O.Policy(O.POLICY_DECODE, 8))
    assert worst < BF16_TOL_SIGMA


def test_config1_bf16_activations_stay_within_their_rounding_noise():
    """With bf16 activations every GEMM operand carries 2^-9 relative rounding
    error, which alone exceeds 2e-2 sigma on the logits: the oracle shows it
    when it rounds to bf16 at the same places.  The CUDA path must not be
    worse than 1.5x that noise."""
    ms, P, G, pol = synth.tiny_shape(), 32, 32, O.Policy(O.POLICY_DECODE, 8)
    W = synth.weights_to_numpy(synth.make_weights(ms, 0, "bfloat16", "cpu"))
    prompt = synth.make_prompt(1, P, 1000, 0)[0]
    exact = O.Sampler(U.oracle_model(ms), W, prompt, G, 1, pol, None, None, "slots", keep_logits=True)
    emul = O.Sampler(U.oracle_model(ms), W, prompt, G, 1, pol, None, None, "slots", rnd=O.round_bf16,
                     keep_logits=True)
    noise = 0.0
    for _ in range(G):
        a = exact.step()
        emul.x[:], emul.M[:] = a.x_in, a.masked_in          # same trajectory for both
        b = emul.step()
        noise = max(noise, np.abs(a.logits - b.logits).max() / a.logits.std())
    worst = run_forced(ms, True, 1, P, G, 1, pol, act=B.DKV_BF16, tol_sigma=1.5 * noise)
    print(f"bf16 activations: oracle rounding noise {noise:.4f} sigma, CUDA {worst:.4f} sigma")
    assert worst <= 1.5 * noise


GQA = dataclasses.replace(synth.tiny_shape(), n_kv_heads=2)


@pytest.mark.parametrize("pol,k,block,order", [
    (O.Policy(O.POLICY_NONE), 2, None, False),
    (O.Policy(O.POLICY_DECODE, 3), 2, 8, False),
    (O.Policy(O.POLICY_DECODE, 0, delay=0), 1, None, False),
    (O.Policy(O.POLICY_PREFILL), 2, None, False),
    (O.Policy(O.POLICY_PD, 4), 2, None, False),
    (O.Policy(O.POLICY_GREEDY, 4, window=4), 1, None, True),
    (O.Policy(O.POLICY_GREEDY, 0, window=2, window_center=O.CENTER_CUR), 2, None, True),
    (O.Policy(O.POLICY_DECODE, 4, shift=1), 2, 8, False),        # shifted outputs (Appendix B, Un-Shift)
    (O.Policy(O.POLICY_PD, 3, shift=1), 1, None, False),
    (O.Policy(O.POLICY_GREEDY, 4, window=4, shift=1), 1, None, True),
    (O.Policy(O.POLICY_DECODE, 4, shift=2), 2, 8, False),        # Appendix B, Un&Right-Shift
    (O.Policy(O.POLICY_PREFILL, shift=2), 1, None, False),
    (O.Policy(O.POLICY_GREEDY, 4, window=2, shift=2), 1, None, True),
    (O.Policy(O.POLICY_PD, 3, isolated_prefill=True), 2, None, False),      # prompt-only prefill pass (Sec. 3.3)
    (O.Policy(O.POLICY_PREFILL, isolated_prefill=True, shift=2), 1, 8, False),
    (O.Policy(O.POLICY_DECODE, 4, score=O.SCORE_MARGIN), 2, None, False),       # other remasking scores (Sec. 3.1)
    (O.Policy(O.POLICY_DECODE, 4, score=O.SCORE_NEG_ENTROPY), 2, 8, False),
])
def test_policies_fp32_batch2_gqa(pol, k, block, order):
    run_forced(GQA, False, 2, 11, 16, k, pol, block, seed=1, with_order=order)


@pytest.mark.parametrize("pol,k", [(O.Policy(O.POLICY_PD, 4), 2), (O.Policy(O.POLICY_GREEDY, 2, window=4), 1),
                                   (O.Policy(O.POLICY_DECODE, 4, shift=1), 2),
                                   (O.Policy(O.POLICY_PD, 3, shift=2), 2),
                                   (O.Policy(O.POLICY_PREFILL, isolated_prefill=True), 2)])
def test_policies_bf16_batch2_gqa(pol, k):
    run_forced(GQA, True, 2, 11, 16, k, pol, None, seed=2, with_order=pol.kind == O.POLICY_GREEDY)


MEDIUM_128 = synth.ModelShape(2, 1024, 8, 2, 128, 1536, 2000, 1999)    # K splits of 4-6, CTA-pair gate/up launch
MEDIUM_64 = synth.ModelShape(2, 768, 12, 4, 64, 1024, 1500, 1499)      # head_dim 64: four heads per weight tile


@pytest.mark.parametrize("fuse", [1, 0])
@pytest.mark.parametrize("ms,pol,k", [(MEDIUM_128, O.Policy(O.POLICY_DECODE, 3), 2),
                                      (MEDIUM_64, O.Policy(O.POLICY_PD, 2), 3),
                                      (MEDIUM_128, O.Policy(O.POLICY_PREFILL, isolated_prefill=True), 2)])
def test_medium_widths_split_k_with_and_without_fused_tails(ms, pol, k, fuse, monkeypatch):
    """Widths at which the projections run with several K splits: with the fused tails (the CTAs of a
    weight tile reduce the splits and apply residual / norm statistics / RoPE / slot scatter themselves)
    and with the switch off (partials to scratch, row kernels), against the oracle, both head paths."""
    monkeypatch.setenv("DKV_FUSE_TAILS", str(fuse))
    worst = run_forced(ms, True, 2, 37, 12 * k, k, pol, 6 * k, seed=5)
    assert worst < BF16_TOL_SIGMA


@pytest.mark.parametrize("fuse", [1, 0])
@pytest.mark.parametrize("ms,pol,k,batch,P", [(MEDIUM_128, O.Policy(O.POLICY_DECODE, 2), 2, 3, 84),
                                              (MEDIUM_64, O.Policy(O.POLICY_PD, 3), 3, 4, 70),
                                              (MEDIUM_64, O.Policy(O.POLICY_NONE), 2, 3, 90),
                                              (MEDIUM_128, O.Policy(O.POLICY_PREFILL, isolated_prefill=True), 2, 5, 60)])
def test_medium_widths_more_than_one_row_tile(ms, pol, k, batch, P, fuse, monkeypatch):
    """Full and refresh steps with more than 256 active rows over several sequences (several row tiles
    per projection, the row kernels behind the multi-tile launches, sequence index and position of
    every row in RoPE and the slot scatter), with the fused tails of the cached steps on and off;
    head_dim 64 and 128, GQA, both head paths, against the oracle."""
    monkeypatch.setenv("DKV_FUSE_TAILS", str(fuse))
    worst = run_forced(ms, True, batch, P, 6 * k, k, pol, None, seed=9)
    assert worst < BF16_TOL_SIGMA


def free_run(ms, bf16, batch, P, G, k, pol, block, seed=0, host=False):
    W, model = U.build_pair(ms, seed, bf16)
    prompts = synth.make_prompt(batch, P, min(1000, ms.vocab - 1), seed)
    x0, m0 = synth.initial_state(prompts, G, ms.mask_id)
    cache = B.dkv_init_cache(model, batch, P + G, P, U.gpu_policy(pol, max_k=k))
    T = G // k
    if host:
        x, m = x0.copy(), m0.copy()
        chosen = np.zeros((T, batch, k), np.int32)
        blk = block or G
        for s in range(T):
            lo = P + (s // (blk // k)) * blk
            B.dkv_step_host(cache, x, m, None, k, lo, lo + blk, G - s * k, chosen[s])
        return W, prompts, x, chosen
    x, m = torch.from_numpy(x0).cuda(), torch.from_numpy(m0).cuda()
    chosen = torch.zeros(T, batch, k, dtype=torch.int32, device="cuda")
    B.dkv_generate(cache, x, m, None, k, block or 0, 0, chosen)
    assert B.dkv_status(cache) == 0
    assert int(m.sum().item()) == 0
    return W, prompts, x.cpu().numpy(), chosen.cpu().numpy()


def test_free_running_generation_fp32_matches_oracle_tokens():
    ms, P, G, k, pol = synth.tiny_shape(), 32, 32, 1, O.Policy(O.POLICY_DECODE, 8)
    W, prompts, x, chosen = free_run(ms, False, 1, P, G, k, pol, None)
    tr = O.generate_one(U.oracle_model(ms), W, prompts[0], G, k, pol)
    ref = O.final_tokens(tr)
    agree = float((x[0] == ref).mean())
    # fp32 against fp64: identical unless a confidence tie is closer than rounding
    assert agree == 1.0, f"token agreement {agree}"
    assert [int(c) for c in chosen[:, 0, 0]] == [s.chosen[0] for s in tr]


def test_free_running_generation_16bit_token_agreement_fraction():
    """16-bit mode, free running (the library picks its own tokens): the fraction of generated
    positions whose final token equals the oracle's.  With random-initialised weights the
    confidences are nearly tied, so the ORDER of unmasking departs from the oracle's within a few
    steps (a 16-bit rounding difference is enough) and later predictions see different contexts;
    the fraction is reported, and only a loose floor is asserted."""
    ms, P, G, k, pol = synth.tiny_shape(), 32, 32, 1, O.Policy(O.POLICY_DECODE, 8)
    fracs = []
    for seed in range(4):
        W, prompts, x, chosen = free_run(ms, True, 1, P, G, k, pol, None, seed=seed)
        tr = O.generate_one(U.oracle_model(ms), W, prompts[0], G, k, pol)
        fracs.append(float((x[0][P:] == O.final_tokens(tr)[P:]).mean()))
    print("16-bit free-running token agreement per seed:", fracs)
    assert np.mean(fracs) >= 0.6


def test_host_driven_steps_equal_device_generation():
    ms, P, G, k, pol = synth.tiny_shape(), 16, 16, 2, O.Policy(O.POLICY_DECODE, 4)
    _, _, xd, cd = free_run(ms, False, 2, P, G, k, pol, 8, seed=3)
    _, _, xh, ch = free_run(ms, False, 2, P, G, k, pol, 8, seed=3, host=True)
    np.testing.assert_array_equal(xd, xh)
    np.testing.assert_array_equal(cd, ch)


def test_interval_one_equals_no_cache_on_the_device():
    ms, P, G = synth.tiny_shape(), 16, 16
    _, _, a, ca = free_run(ms, True, 1, P, G, 1, O.Policy(O.POLICY_NONE), None, seed=4)
    _, _, b, cb = free_run(ms, True, 1, P, G, 1, O.Policy(O.POLICY_DECODE, 1), None, seed=4)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(ca, cb)


def test_explicit_refresh_recomputes_everything():
    ms = synth.tiny_shape()
    W, model = U.build_pair(ms, 5, False)
    P, G = 8, 8
    pol = O.Policy(O.POLICY_DECODE, 0)
    cache = B.dkv_init_cache(model, 1, P + G, P, U.gpu_policy(pol))
    x, m = synth.random_mask_state(1, P, G, 3, ms.mask_id, 5)
    x[m == 1] = ms.mask_id
    tx, tm = torch.from_numpy(x).cuda(), torch.from_numpy(m).cuda()
    conf = torch.empty(1, P + G, device="cuda")
    pred = torch.empty(1, P + G, dtype=torch.int32, device="cuda")
    nh = int(m.sum())
    logits = torch.zeros(G, ms.vocab, device="cuda")
    B.dkv_step(cache, tx, tm, None, 1, P, P + G, nh, conf, pred, logits)       # step 1: full
    B.dkv_step(cache, tx, tm, None, 1, P, P + G, nh, conf, pred, logits)       # cached
    B.dkv_refresh(cache, B.DKV_REFRESH_ALL)
    B.dkv_step(cache, tx, tm, None, 1, P, P + G, nh, conf, pred, logits)       # forced full
    prov = torch.empty(1, P + G, dtype=torch.int32, device="cuda")
    B.dkv_get_provenance(cache, prov)
    assert (prov.cpu().numpy() == 3).all()
    ref = O.vanilla_forward(U.oracle_model(ms), W, x[0].astype(np.int64))[np.nonzero(m[0])[0]]
    assert np.abs(logits[:nh].cpu().numpy() - ref).max() < F32_TOL


def test_argument_errors_are_status_codes():
    ms = synth.tiny_shape()
    _, model = U.build_pair(ms, 0, False)
    with pytest.raises(B.DkvError) as e:
        B.dkv_init_cache(model, 1, 8, 9, B.make_policy(B.DKV_POLICY_DECODE))
    assert e.value.status == -2
    cache = B.dkv_init_cache(model, 1, 16, 8, B.make_policy(B.DKV_POLICY_GREEDY, window=4))
    x = torch.zeros(1, 16, dtype=torch.int32, device="cuda")
    m = torch.zeros(1, 16, dtype=torch.uint8, device="cuda")
    conf = torch.empty(1, 16, device="cuda")
    pred = torch.empty(1, 16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DkvError) as e:
        B.dkv_step(cache, x, m, None, 1, 8, 16, 8, conf, pred)          # Greedy without next_pos
    assert e.value.status == -1
    with pytest.raises(B.DkvError) as e:
        B.dkv_step(cache, x, m, x, 3, 8, 16, 8, conf, pred)             # k > max_k
    assert e.value.status == -2
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.DkvError) as e:
        B.dkv_init_cache(model, 1, 16, 8, B.make_policy(B.DKV_POLICY_DECODE), arena=small)
    assert e.value.status == -4


@pytest.mark.parametrize("score", [O.SCORE_MAXPROB, O.SCORE_MARGIN, O.SCORE_NEG_ENTROPY])
@pytest.mark.parametrize("vocab", [1024, 1000, 4129])
def test_fused_head_statistics_match_materialised_logits(vocab, score):
    """Without a logits buffer the head GEMM's epilogue reduces the vocabulary
    to (max, argmax, sum exp) itself; with one, the logits are written and a
    separate kernel reduces them.  Both must give the same confidences and
    tokens, and the oracle's (ragged vocabulary sizes included)."""
    ms = dataclasses.replace(synth.tiny_shape(), vocab=vocab, mask_id=vocab - 1)
    W, model = U.build_pair(ms, 7, True)
    P, G = 16, 48
    x, m = synth.random_mask_state(2, P, G, 9, ms.mask_id, 7)
    tx, tm = torch.from_numpy(x).cuda(), torch.from_numpy(m).cuda()
    out = []
    for with_logits in (False, True):
        cache = B.dkv_init_cache(model, 2, P + G, P, B.make_policy(B.DKV_POLICY_DECODE, 4, score=score))
        conf = torch.empty(2, P + G, device="cuda")
        pred = torch.empty(2, P + G, dtype=torch.int32, device="cuda")
        logits = torch.zeros(2 * G, vocab, device="cuda") if with_logits else None
        B.dkv_step(cache, tx, tm, None, 1, P, P + G, int(m.sum(1).max()), conf, pred, logits)
        assert B.dkv_status(cache) == 0
        out.append((conf.cpu().numpy(), pred.cpu().numpy()))
    (cf, pf), (cu, pu) = out
    head = m.astype(bool)
    np.testing.assert_array_equal(pf, pu)
    np.testing.assert_allclose(cf[head], cu[head], rtol=5e-5, atol=2e-8)
    assert np.isneginf(cf[~head]).all() and (pf[~head] == -1).all()
    for b in range(2):
        ref = O.vanilla_forward(U.oracle_model(ms), W, x[b].astype(np.int64))
        for pos in np.nonzero(m[b])[0]:
            c, p = O.confidence(ref[pos], ms.mask_id, score)
            top2 = np.sort(np.delete(ref[pos], ms.mask_id))[-2:]
            if top2[1] - top2[0] > 4e-2 * ref[pos].std():
                assert pf[b, pos] == p
            if score == O.SCORE_MARGIN:      # a difference of two probabilities of about 1/vocab
                assert abs(cf[b, pos] - c) < 0.1 / vocab
            else:
                assert abs(cf[b, pos] - c) < 0.05 * abs(c)
