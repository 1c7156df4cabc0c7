"""Helpers shared by the GPU parity tests: build the same seeded model for the
oracle (numpy) and for the CUDA library, and drive both over one trajectory."""
from __future__ import annotations

import numpy as np
import torch

from oracle import dkv_oracle as O
from paper_2505_15781_b200 import binding as B
from paper_2505_15781_b200 import synth

POLICY_KIND = {O.POLICY_NONE: B.DKV_POLICY_NONE, O.POLICY_DECODE: B.DKV_POLICY_DECODE,
               O.POLICY_PREFILL: B.DKV_POLICY_PREFILL, O.POLICY_PD: B.DKV_POLICY_PD,
               O.POLICY_GREEDY: B.DKV_POLICY_GREEDY}


def oracle_model(ms: synth.ModelShape) -> O.Model:
    return O.Model(ms.n_layers, ms.d_model, ms.n_q_heads, ms.n_kv_heads, ms.head_dim, ms.d_ffn, ms.vocab,
                   ms.mask_id, ms.rope_theta, ms.rms_eps)


def build_pair(ms: synth.ModelShape, seed: int, bf16: bool, oracle_dtype=np.float64, gen_device="cuda", act=None):
    """(oracle weights as numpy, CUDA model handle).  In bf16 mode the oracle
    gets the bf16-rounded values upcast, i.e. the same numbers.  act: the
    activation / cache type of the CUDA model (default: fp16 with bf16
    weights, the benchmark's configuration)."""
    w = synth.make_weights(ms, seed, "bfloat16" if bf16 else "float32", gen_device)
    W = synth.weights_to_numpy(w, oracle_dtype)
    wd = {k: (v.cuda() if k != "layers" else [{kk: vv.cuda() for kk, vv in lw.items()} for lw in v])
          for k, v in w.items()}
    model = B.dkv_model_create(ms, wd, B.DKV_BF16 if bf16 else B.DKV_F32, act)
    return W, model


def gpu_policy(pol: O.Policy, max_head_rows=0, max_k=1):
    return B.make_policy(POLICY_KIND[pol.kind], pol.refresh_interval, pol.delay, pol.window,
                         B.DKV_CENTER_PREV if pol.window_center == O.CENTER_PREV else B.DKV_CENTER_CUR,
                         max_head_rows, max_k, pol.shift, pol.score, int(pol.isolated_prefill))


class ForcedRun:
    """Feeds the oracle's (x_t, M_t) of every step to the CUDA library and
    collects what it returns."""

    def __init__(self, ms, model, batch, P, G, pol: O.Policy, k, fused=False, arena_fill=None):
        """fused: also drive a second handle WITHOUT a logits buffer, i.e. through the head GEMM's
        statistics epilogue (the path the benchmark times); its conf / pred land in conf_f / pred_f.
        arena_fill: byte value the arenas are filled with before dkv_init_cache (None: torch.empty)."""
        self.ms, self.B, self.L, self.P, self.k, self.score = ms, batch, P + G, P, k, pol.score
        dev = "cuda"

        def arena():
            if arena_fill is None:
                return None
            need = B.dkv_cache_bytes(model, batch, P + G, gpu_policy(pol, max_k=k))
            return torch.full((need + 256,), arena_fill, dtype=torch.uint8, device=dev)
        self.cache = B.dkv_init_cache(model, batch, P + G, P, gpu_policy(pol, max_k=k), arena=arena())
        self.cache_f = B.dkv_init_cache(model, batch, P + G, P, gpu_policy(pol, max_k=k), arena=arena()) if fused else None
        self.conf_f = torch.empty(batch, self.L, dtype=torch.float32, device=dev)
        self.pred_f = torch.empty(batch, self.L, dtype=torch.int32, device=dev)
        self.conf = torch.empty(batch, self.L, dtype=torch.float32, device=dev)
        self.pred = torch.empty(batch, self.L, dtype=torch.int32, device=dev)
        self.logits = torch.zeros(batch * G, ms.vocab, dtype=torch.float32, device=dev)
        self.act_idx = torch.empty(batch * self.L, dtype=torch.int32, device=dev)
        self.row_off = torch.empty(batch + 1, dtype=torch.int32, device=dev)
        self.inv = torch.empty(batch, self.L, dtype=torch.int32, device=dev)
        self.prov = torch.empty(batch, self.L, dtype=torch.int32, device=dev)

    def step(self, traces_t, greedy: bool):
        """traces_t: list over sequences of the oracle's StepTrace for this step."""
        x = torch.tensor(np.stack([s.x_in for s in traces_t]), dtype=torch.int32, device="cuda")
        m = torch.tensor(np.stack([s.masked_in for s in traces_t]), dtype=torch.uint8, device="cuda")
        npos = None
        if greedy:
            npos = torch.tensor(np.stack([np.array(s.chosen) for s in traces_t]), dtype=torch.int32, device="cuda")
        lo, hi = traces_t[0].cand
        rows_bound = int(max(s.masked_in.sum() for s in traces_t))
        B.dkv_step(self.cache, x, m, npos, self.k, lo, hi, rows_bound, self.conf, self.pred, self.logits)
        if self.cache_f is not None:
            B.dkv_step(self.cache_f, x, m, npos, self.k, lo, hi, rows_bound, self.conf_f, self.pred_f, None)
        B.dkv_get_index_maps(self.cache, self.act_idx, self.row_off, self.inv)
        B.dkv_get_provenance(self.cache, self.prov)
        torch.cuda.synchronize()
        return x, m


def score_bound(score, eps, conf_ref, p_max):
    """How far a score may move when every logit moves by at most eps.  With |dl_i| <= eps every
    probability moves by a factor within [e^-2eps, e^2eps] (numerator and normaliser each by e^eps):
    the largest probability by (e^2eps - 1) p_max; the margin of the two largest (order statistics are
    1-Lipschitz in the sup norm) by twice that; sum p log p by 2 eps + (e^2eps - 1) |sum p log p|."""
    g = np.expm1(2.0 * eps)
    if score == O.SCORE_MAXPROB:
        return g * p_max
    if score == O.SCORE_MARGIN:
        return 2.0 * g * p_max
    return 2.0 * eps + g * abs(conf_ref)


def check_head_outputs(conf, pred, s, mask_id, score, eps, what):
    """conf / pred of one sequence against the oracle's trace s, given that the logits are within
    eps (absolute) of the oracle's: the token must agree wherever the oracle's two largest logits are
    more than 2 eps apart, the score within score_bound (plus fp32 evaluation noise)."""
    for j, pos in enumerate(s.head_rows):
        l = np.array(s.logits[j], dtype=np.float64)
        l[mask_id] = -np.inf
        top2 = np.sort(l)[-2:]
        if top2[1] - top2[0] > 2.0 * eps:
            assert pred[pos] == s.pred[pos], f"{what}: token at position {pos}, step {s.t}"
        p_max = 1.0 / np.exp(l - top2[1]).sum()
        bound = score_bound(score, eps, s.conf[pos], p_max) + 1e-5 * abs(s.conf[pos]) + 1e-9
        assert abs(conf[pos] - s.conf[pos]) <= bound, \
            f"{what}: score at position {pos}, step {s.t}: {conf[pos]} vs {s.conf[pos]} (bound {bound})"


def compare_step(run: ForcedRun, traces_t, greedy, logit_tol_abs=None, logit_tol_sigma=None):
    """Integer outputs bit-exact; logits within the given tolerance; with a sigma tolerance (16-bit
    modes) also the scores and tokens of the head rows, within what that logit tolerance allows, on
    the materialised-logits path and, when the run drives one, on the fused head path.  Returns
    (max abs logit error, sigma of the oracle's logits, conf, pred)."""
    x, m = run.step(traces_t, greedy)
    L = run.L
    row_off = run.row_off.cpu().numpy()
    act = run.act_idx.cpu().numpy()
    inv = run.inv.cpu().numpy()
    prov = run.prov.cpu().numpy()
    conf = run.conf.cpu().numpy()
    pred = run.pred.cpu().numpy()
    n_head = sum(len(s.head_rows) for s in traces_t)
    logits = run.logits[:n_head].cpu().numpy()
    max_err, sig, hoff = 0.0, 1.0, 0
    ref_all = np.concatenate([s.logits for s in traces_t], axis=0) if traces_t[0].logits is not None else None
    if ref_all is not None and len(ref_all):
        sig = float(ref_all.std())
    for b, s in enumerate(traces_t):
        got = act[row_off[b]:row_off[b + 1]]
        np.testing.assert_array_equal(got, s.active + b * L, err_msg=f"active set, step {s.t}, seq {b}")
        exp_inv = np.full(L, -1)
        exp_inv[s.active] = np.arange(len(s.active)) + row_off[b]
        np.testing.assert_array_equal(inv[b], exp_inv)
        np.testing.assert_array_equal(prov[b], s.written_step, err_msg=f"provenance, step {s.t}")
        nh = len(s.head_rows)
        if s.logits is not None and nh:
            err = np.abs(logits[hoff:hoff + nh] - s.logits).max()
            max_err = max(max_err, float(err))
        hoff += nh
        # conf / pred at original positions; -inf / -1 elsewhere
        not_head = np.ones(L, bool)
        not_head[s.head_rows] = False
        assert np.isneginf(conf[b][not_head]).all() and (pred[b][not_head] == -1).all()
    if logit_tol_abs is not None:
        assert max_err <= logit_tol_abs, f"step {traces_t[0].t}: logits max-abs error {max_err} > {logit_tol_abs}"
    if logit_tol_sigma is not None:
        assert max_err <= logit_tol_sigma * sig, \
            f"step {traces_t[0].t}: logits max-abs error {max_err} > {logit_tol_sigma} * sigma ({sig})"
        if ref_all is not None:
            eps = logit_tol_sigma * sig
            conf_f, pred_f = run.conf_f.cpu().numpy(), run.pred_f.cpu().numpy()
            for b, s in enumerate(traces_t):
                check_head_outputs(conf[b], pred[b], s, run.ms.mask_id, run.score, eps, "materialised logits")
                if run.cache_f is not None:
                    check_head_outputs(conf_f[b], pred_f[b], s, run.ms.mask_id, run.score, eps, "fused head epilogue")
                    not_head = np.ones(L, bool)
                    not_head[s.head_rows] = False
                    assert np.isneginf(conf_f[b][not_head]).all() and (pred_f[b][not_head] == -1).all()
    return max_err, sig, conf, pred
