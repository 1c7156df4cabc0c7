"""Seeded random configurations of small models through the whole step path, against the oracle:
shapes (widths that are not multiples of the GEMM tiles, GQA groups, head_dim 64 and 128, odd
lengths), batch, tokens per step, blocks and every policy, in the fp32 check mode and in the 16-bit
mode.  Each case is a handful of steps; integers are compared bit for bit, logits within the stated
tolerances."""
import numpy as np
import pytest

from oracle import dkv_oracle as O
from paper_2505_15781_b200 import binding as B
from paper_2505_15781_b200 import synth
from tests import gpu_util as U
from tests.test_gpu_step import run_forced

pytestmark = pytest.mark.gpu


def random_case(seed):
    r = np.random.Generator(np.random.PCG64(9000 + seed))
    head_dim = int(r.choice([64, 128]))
    n_kv = int(r.choice([1, 2, 3]))
    group = int(r.choice([1, 2, 4]))
    n_q = n_kv * group
    d_model = int(r.choice([192, 256, 320]))
    d_ffn = int(r.choice([256, 384, 688]))           # 688 is no multiple of 128: no fused SwiGLU layout there
    vocab = int(r.choice([515, 1000, 1024]))
    ms = synth.ModelShape(int(r.integers(1, 4)), d_model, n_q, n_kv, head_dim, d_ffn, vocab, vocab - 1)
    batch = int(r.integers(1, 4))
    k = int(r.choice([1, 2, 3]))
    T = int(r.integers(3, 7))
    G = k * T
    block = None
    if T % 2 == 0 and r.random() < 0.5:
        block = G // 2
    P = int(r.integers(0, 40)) if r.random() < 0.8 else 0
    kind = int(r.choice([O.POLICY_NONE, O.POLICY_DECODE, O.POLICY_PREFILL, O.POLICY_PD, O.POLICY_GREEDY]))
    shift = int(r.choice([0, 0, 1, 2])) if P >= 1 else 0
    pol = O.Policy(kind, int(r.integers(0, 4)), delay=int(r.choice([1, 1, 0])), window=int(r.integers(0, 5)),
                   window_center=int(r.choice([O.CENTER_PREV, O.CENTER_CUR])), shift=shift,
                   score=int(r.choice([O.SCORE_MAXPROB, O.SCORE_MARGIN, O.SCORE_NEG_ENTROPY])),
                   isolated_prefill=bool(kind in (O.POLICY_PREFILL, O.POLICY_PD) and P > 0 and r.random() < 0.4))
    if kind == O.POLICY_GREEDY:
        block = None
    return ms, batch, P, G, k, pol, block


@pytest.mark.parametrize("seed", range(40))
def test_random_configuration_fp32(seed):
    ms, batch, P, G, k, pol, block = random_case(seed)
    run_forced(ms, False, batch, P, G, k, pol, block, seed=seed, with_order=pol.kind == O.POLICY_GREEDY)


@pytest.mark.parametrize("seed", range(40, 64))
def test_random_configuration_16bit(seed):
    ms, batch, P, G, k, pol, block = random_case(seed)
    run_forced(ms, True, batch, P, G, k, pol, block, seed=seed, with_order=pol.kind == O.POLICY_GREEDY)


def medium_case(seed):
    """Widths at which the projections take several K splits (the fused cross-CTA tails), GQA groups up
    to 7, head_dim 64 and 128, d_ffn with and without the CTA-pair launch, up to a few hundred rows."""
    r = np.random.Generator(np.random.PCG64(777 + seed))
    hd = int(r.choice([64, 128]))
    n_kv = int(r.choice([1, 2, 4]))
    group = int(r.choice([1, 2, 4, 7]))
    d_model = int(r.choice([512, 768, 1024, 1536, 2048]))
    d_ffn = int(r.choice([512, 1024, 1280, 1536, 2816, 4096]))
    vocab = int(r.choice([1000, 2048, 5000]))
    ms = synth.ModelShape(int(r.integers(1, 3)), d_model, n_kv * group, n_kv, hd, d_ffn, vocab, vocab - 1)
    batch = int(r.integers(1, 4))
    k = int(r.choice([1, 2]))
    G = k * int(r.integers(2, 5)) * int(r.choice([1, 8, 20]))
    P = int(r.integers(0, 120))
    kind = int(r.choice([O.POLICY_NONE, O.POLICY_DECODE, O.POLICY_PREFILL, O.POLICY_PD, O.POLICY_GREEDY]))
    pol = O.Policy(kind, int(r.integers(0, 4)), delay=int(r.choice([1, 1, 0])), window=int(r.integers(0, 5)),
                   shift=int(r.choice([0, 0, 1])) if P >= 1 else 0, score=int(r.choice([0, 1, 2])),
                   isolated_prefill=bool(kind in (O.POLICY_PREFILL, O.POLICY_PD) and P > 0 and r.random() < 0.4))
    return ms, batch, P, G, k, pol


@pytest.mark.parametrize("seed", range(24))
def test_random_medium_configuration_16bit_first_steps(seed):
    """The first four steps of a random medium-width configuration against the oracle, logits within
    2e-2 sigma, integers bit for bit, scores and tokens on both head paths."""
    ms, batch, P, G, k, pol = medium_case(seed)
    greedy = pol.kind == O.POLICY_GREEDY
    W, model = U.build_pair(ms, seed, True)
    order = synth.random_order(batch, P, G, k, seed) if greedy else None
    prompts = synth.make_prompt(batch, P, min(1000, ms.vocab - 1), seed)
    samplers = [O.Sampler(U.oracle_model(ms), W, prompts[b], G, k, pol, None, order[:, b, :] if greedy else None,
                          "slots" if greedy else "literal", keep_logits=True) for b in range(batch)]
    run = U.ForcedRun(ms, model, batch, P, G, pol, k, fused=True)
    for _ in range(min(G // k, 4)):
        U.compare_step(run, [s.step() for s in samplers], greedy, logit_tol_sigma=2e-2)
    assert B.dkv_status(run.cache) == 0 and B.dkv_status(run.cache_f) == 0
