"""CPU oracle for the dKV-Cache denoising step (test infrastructure).

This file is TEST INFRASTRUCTURE.  It is a plain, slow numpy restatement of
what the paper's method computes, written to be checked against the paper by
eye.  Only the test-suite, the smoke check and the benchmark's CPU-baseline
leg may import it; the CUDA library never does, and the two share no code.

What follows what (the paper: "dKV-Cache: The Cache for Diffusion Language
Models"):

* ``attention``            Eq. 1 / Eq. 4: softmax(Q K^T / sqrt(d_k)) V, no mask.
* ``active_set``           Eq. 4 (Decode: rows M_{t-1}), Eq. 3 (delay 0: rows
                           M_t), the refresh paragraph of Sec. 3.3, the
                           Prefill / PD paragraph, Sec. 3.4 (Greedy + window).
* ``concat_reorder_maps``  Appendix A: the two physical orders and the map I'.
* ``LiteralCache.step``    Sec. 3.3 / Appendix A / Algorithm 1: the cache as physically
                           ordered arrays (cached rows, then fresh rows), narrowed
                           through index maps, concatenated for the attention of Eq. 4.
* ``SlotCache.step``       the same step written with position-addressed
                           slots; ``tests`` check literal == slots.
* ``select_unmask``        Sec. 3.1, "keeping the most confident ones".
* ``Sampler`` / ``generate_one``  the sampling loop of Sec. 3.1 (``Policy.shift``: Appendix B, Un-Shift and Un&Right-Shift) with semi-AR blocks
                           (Table 4 of the appendix: L, T, block size).
* ``cache_ratio``          the cache-ratio metric of Sec. 4.1.

Model architecture (the paper only says "transformer, with or without GQA"):
pre-norm residual blocks, RMSNorm, rotate-half RoPE on absolute positions,
SwiGLU, no biases, no attention mask, untied head.

Parity status: everything here is pinned by ``tests/test_oracle_*.py`` except
generation QUALITY (accuracy on benchmarks), which needs trained weights and
is "parity unpinned".
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

POLICY_NONE, POLICY_DECODE, POLICY_PREFILL, POLICY_PD, POLICY_GREEDY = 0, 1, 2, 3, 4
CENTER_PREV, CENTER_CUR = 0, 1


@dataclasses.dataclass(frozen=True)
class Policy:
    kind: int = POLICY_DECODE
    refresh_interval: int = 0      # N; 0 = never after step 1
    delay: int = 1                 # 1 = one-step delayed caching (Eq. 4); 0 = Eq. 3
    window: int = 0                # w of Sec. 3.4
    window_center: int = CENTER_PREV
    isolated_prefill: bool = False  # Prefill / PD only: at step 1 the prompt rows are computed alone (they attend
                                   #    to prompt slots only), then the generation rows over all slots (Sec. 3.3:
                                   #    prefill tokens mostly attend to each other; prefill/decode disaggregation)
    shift: int = 0                 # 1: the logits of position j are read at row j-1 (Appendix B, Un-Shift)
                                   # 2: the same, and a row is cached only once its input AND the token it
                                   #    predicts are decoded (Appendix B, Un&Right-Shift)
    score: int = 0                 # SCORE_*: what the top-k selection ranks (Sec. 3.1)


@dataclasses.dataclass(frozen=True)
class Model:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    mask_id: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5


# ---------------------------------------------------------------------------
# building blocks
# ---------------------------------------------------------------------------

def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even); result in a's dtype."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).astype(a.dtype).reshape(a.shape)


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate-half RoPE.  x: [n, heads, d_h]; pos: [n] absolute positions."""
    d_h = x.shape[-1]
    half = d_h // 2
    inv_freq = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / d_h)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]
    c = np.cos(ang).astype(x.dtype)[:, None, :]
    s = np.sin(ang).astype(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """q: [n, H_q, d_h]; k, v: [m, H_kv, d_h].  Every query attends to every
    key (no mask).  Query head h uses key/value head h // (H_q / H_kv)."""
    n, hq, dh = q.shape
    hkv = k.shape[1]
    group = hq // hkv
    out = np.empty_like(q)
    for h in range(hq):
        kh = k[:, h // group, :]
        vh = v[:, h // group, :]
        s = (q[:, h, :] @ kh.T) / math.sqrt(dh)
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=-1, keepdims=True)
        out[:, h, :] = p @ vh
    return out


# ---------------------------------------------------------------------------
# policy: which rows are recomputed at step t
# ---------------------------------------------------------------------------

def is_refresh_step(t: int, pol: Policy) -> bool:
    """t is 1-based.  Step 1 is always a full step.  With interval N the
    0-based step s = t-1 refreshes when s mod N == 0."""
    if pol.kind == POLICY_NONE or t == 1:
        return True
    if pol.kind == POLICY_PREFILL:
        return False
    return pol.refresh_interval > 0 and (t - 1) % pol.refresh_interval == 0


def greedy_window(centers: Sequence[int], w: int, L: int) -> List[int]:
    out = set()
    for c in centers:
        lo = c - int(math.ceil(w / 2.0))
        hi = c + int(math.floor(w / 2.0))
        out.update(i for i in range(lo, hi + 1) if 0 <= i < L)
    return sorted(out)


def active_set(t: int, pol: Policy, L: int, P: int, M_prev: Optional[np.ndarray],
               M_cur: np.ndarray, D_cur: Optional[Sequence[int]] = None,
               D_prev: Optional[Sequence[int]] = None, force_refresh: bool = False) -> np.ndarray:
    """Ascending positions whose Q/K/V/FFN are recomputed at step t.
    M_prev / M_cur: uint8 [L] mask bitmaps of steps t-1 and t (1 = masked)."""
    everything = np.arange(L, dtype=np.int64)
    if pol.kind == POLICY_NONE or t == 1:
        return everything
    refresh = force_refresh or is_refresh_step(t, pol)
    if pol.kind == POLICY_PREFILL:
        return np.arange(P, L, dtype=np.int64)
    if pol.kind == POLICY_PD and refresh:
        return np.arange(P, L, dtype=np.int64)
    if refresh:
        return everything
    if pol.kind in (POLICY_DECODE, POLICY_PD):
        src = M_prev if pol.delay == 1 else M_cur
        return np.nonzero(src)[0].astype(np.int64)
    if pol.kind == POLICY_GREEDY:
        d_cur = list(D_cur) if D_cur is not None else []
        d_prev = list(D_prev) if D_prev is not None else []
        centers = d_prev if pol.window_center == CENTER_PREV else d_cur
        rows = set(d_cur) | set(d_prev) | set(greedy_window(centers, pol.window, L))
        return np.array(sorted(rows), dtype=np.int64)
    raise ValueError("unknown policy")


def concat_reorder_maps(cached_prev: Sequence[int], active_prev: Sequence[int],
                        cached_next: Sequence[int], active_next: Sequence[int]):
    """Appendix A.  Physical order at one step is [cached ; active]; returns
    (order_prev, order_next, full_map, cache_entries) where full_map[j] is the
    index inside order_prev of order_next[j] and cache_entries is its prefix
    for the next cached set."""
    order_prev = list(cached_prev) + list(active_prev)
    order_next = list(cached_next) + list(active_next)
    where = {p: j for j, p in enumerate(order_prev)}
    full_map = [where[p] for p in order_next]
    return order_prev, order_next, full_map, full_map[:len(cached_next)]


# ---------------------------------------------------------------------------
# transformer on a subset of rows
# ---------------------------------------------------------------------------

def _identity(a):
    return a


class _Forward:
    """Row-wise parts of one decoder layer, shared by the two cache forms.
    ``rnd`` is the identity, or ``round_bf16`` to emulate where a bf16
    tensor-core pipeline rounds its MMA operands."""

    def __init__(self, model: Model, W: Dict, rnd=_identity):
        self.m, self.W, self.rnd = model, W, rnd

    def embed(self, tokens_rows: np.ndarray) -> np.ndarray:
        return self.W["embed"][tokens_rows]

    def qkv(self, l: int, h: np.ndarray, pos: np.ndarray):
        m, lw = self.m, self.W["layers"][l]
        n = self.rnd(rmsnorm(h, lw["attn_norm"], m.rms_eps))
        q = (n @ lw["wq"].T).reshape(-1, m.n_q_heads, m.head_dim)
        k = (n @ lw["wk"].T).reshape(-1, m.n_kv_heads, m.head_dim)
        v = (n @ lw["wv"].T).reshape(-1, m.n_kv_heads, m.head_dim)
        q = self.rnd(rope(q, pos, m.rope_theta))
        k = self.rnd(rope(k, pos, m.rope_theta))
        return q, k, self.rnd(v)

    def after_attention(self, l: int, h: np.ndarray, a: np.ndarray) -> np.ndarray:
        m, lw = self.m, self.W["layers"][l]
        h = h + self.rnd(a.reshape(a.shape[0], -1)) @ lw["wo"].T
        n2 = self.rnd(rmsnorm(h, lw["ffn_norm"], m.rms_eps))
        u = self.rnd(silu(n2 @ lw["wg"].T) * (n2 @ lw["wu"].T))
        return h + u @ lw["wd"].T

    def logits(self, h: np.ndarray) -> np.ndarray:
        n = self.rnd(rmsnorm(h, self.W["final_norm"], self.m.rms_eps))
        return n @ self.W["head"].T


def vanilla_forward(model: Model, W: Dict, x: np.ndarray, rnd=_identity) -> np.ndarray:
    """Full bidirectional forward of one sequence x [L] -> logits [L, V]."""
    fw = _Forward(model, W, rnd)
    pos = np.arange(len(x))
    h = fw.embed(x)
    for l in range(model.n_layers):
        q, k, v = fw.qkv(l, h, pos)
        h = fw.after_attention(l, h, attention(q, k, v))
    return fw.logits(h)


def _scatter_logits(fw: "_Forward", h: np.ndarray, A: np.ndarray, logit_rows, L: int) -> "SparseLogits":
    """Logits of the wanted rows, addressed by ORIGINAL position (the scatter that ends Algorithm 1)."""
    if logit_rows is None:
        sel = np.arange(len(A))
    else:
        where = {int(p): j for j, p in enumerate(A)}
        sel = np.array([where[int(p)] for p in logit_rows], dtype=np.int64)
    return SparseLogits(A[sel], fw.logits(h[sel]) if len(sel) else np.zeros((0, fw.m.vocab)), L)


def prompt_only_kv(fw: "_Forward", x_prompt: np.ndarray):
    """K/V of every layer for a prompt evaluated ALONE (its rows attend to each
    other and to nothing else): the prefill phase of a disaggregated
    prefill / decode deployment (Sec. 3.3).  Returns [(k_l, v_l)] per layer."""
    pos = np.arange(len(x_prompt))
    h = fw.embed(x_prompt)
    out = []
    for l in range(fw.m.n_layers):
        q, k, v = fw.qkv(l, h, pos)
        out.append((k, v))
        h = fw.after_attention(l, h, attention(q, k, v))
    return out


class SparseLogits:
    """Logits scattered back to the original positions: indexable by position
    (a row of NaN where no logits were computed)."""

    def __init__(self, positions: np.ndarray, rows: np.ndarray, L: int):
        self.positions, self.rows, self.L = np.asarray(positions, dtype=np.int64), rows, L
        self._where = {int(p): j for j, p in enumerate(self.positions)}

    def __getitem__(self, idx):
        if np.isscalar(idx) or isinstance(idx, (int, np.integer)):
            j = self._where.get(int(idx))
            return self.rows[j] if j is not None else np.full(self.rows.shape[1], np.nan)
        return np.stack([self[int(i)] for i in np.asarray(idx).ravel()]) if len(np.asarray(idx).ravel()) else \
            np.zeros((0, self.rows.shape[1]))

    def dense(self) -> np.ndarray:
        out = np.full((self.L, self.rows.shape[1]), np.nan, dtype=self.rows.dtype)
        out[self.positions] = self.rows
        return out


class LiteralCache:
    """The cache as Sec. 3.3 and Appendix A describe it: per layer a pair of
    arrays whose rows sit in a PHYSICAL order (``self.order`` lists the position
    each physical row belongs to), cached rows first, the rows computed in the
    last evaluation behind them.  Nothing is addressed by position: a step
    first narrows the arrays to the rows it will serve from the cache, appends
    the freshly computed rows (Eq. 4: K of the cached set next to K of the
    active set), attends over the concatenation, and finally narrows again to
    what the following step may reuse.  Narrowing goes through an index map
    into the current physical order (the map I' of Appendix A)."""

    def __init__(self, model: Model, W: Dict, L: int, rnd=_identity):
        self.fw = _Forward(model, W, rnd)
        self.m, self.L = model, L
        self.order: List[int] = []                 # position of each physical row
        self.K: List[Optional[np.ndarray]] = [None] * model.n_layers
        self.V: List[Optional[np.ndarray]] = [None] * model.n_layers
        self.written_step = np.zeros(L, dtype=np.int64)
        self.t = 0

    def prefill(self, x_prompt: np.ndarray):
        """Hold the K/V of a prompt evaluated alone, stamped with the step that follows."""
        P = len(x_prompt)
        kv = prompt_only_kv(self.fw, np.asarray(x_prompt))
        for l, (k, v) in enumerate(kv):
            self.K[l], self.V[l] = k, v
        self.order = list(range(P))
        self.written_step[:P] = self.t + 1

    def narrow_to(self, keep: Sequence[int]):
        """Physical rows become exactly the positions ``keep``, in that order
        (gather through the index map into the present order)."""
        present = {p: j for j, p in enumerate(self.order)}
        imap = np.array([present[p] for p in keep], dtype=np.int64)
        for l in range(self.m.n_layers):
            if self.K[l] is not None:
                self.K[l], self.V[l] = self.K[l][imap], self.V[l][imap]
        self.order = list(keep)

    def step(self, x: np.ndarray, A: np.ndarray, keep_after: Optional[Sequence[int]] = None,
             logit_rows: Optional[Sequence[int]] = None):
        """One model evaluation in which the rows A (ascending positions) are
        recomputed and every other position is served from the cache.
        keep_after: the positions the following step will serve from the cache,
        when already known (None keeps every row).  logit_rows: positions (a
        subset of A) whose logits are wanted; the head is row-wise, so leaving
        the other rows out changes nothing for these (None = all of A).
        Returns the logits addressed by ORIGINAL position."""
        self.t += 1
        m, L = self.m, self.L
        A = np.asarray(A, dtype=np.int64)
        recomputed = set(A.tolist())
        stable = [p for p in range(L) if p not in recomputed]     # served from the cache this step
        absent = sorted(set(stable) - set(self.order))
        if absent:
            raise KeyError(f"step {self.t}: cached K/V missing for positions {absent[:8]}")
        self.narrow_to(stable)
        h = self.fw.embed(x[A])
        for l in range(m.n_layers):
            # rotary phases follow the rows' original positions, whatever their physical place
            q, k_new, v_new = self.fw.qkv(l, h, A)
            if stable:
                self.K[l] = np.concatenate([self.K[l], k_new], axis=0)
                self.V[l] = np.concatenate([self.V[l], v_new], axis=0)
            else:
                self.K[l], self.V[l] = k_new, v_new
            h = self.fw.after_attention(l, h, attention(q, self.K[l], self.V[l]))
        self.order = stable + A.tolist()
        self.written_step[A] = self.t
        if keep_after is not None:
            self.narrow_to(list(keep_after))
        return _scatter_logits(self.fw, h, A, logit_rows, L)


class SlotCache:
    """The same step with position-addressed slots: every active row writes
    its fresh K/V into its own slot, then attention reads all L slots."""

    def __init__(self, model: Model, W: Dict, L: int, rnd=_identity, dtype=np.float64):
        self.fw = _Forward(model, W, rnd)
        self.m, self.L = model, L
        shp = (model.n_layers, L, model.n_kv_heads, model.head_dim)
        self.K = np.full(shp, np.nan, dtype=dtype)
        self.V = np.full(shp, np.nan, dtype=dtype)
        self.written_step = np.zeros(L, dtype=np.int64)
        self.t = 0

    def prefill(self, x_prompt: np.ndarray):
        """Fill the prompt's slots with its K/V evaluated alone, stamped with the step that follows."""
        P = len(x_prompt)
        for l, (k, v) in enumerate(prompt_only_kv(self.fw, np.asarray(x_prompt))):
            self.K[l, :P] = k
            self.V[l, :P] = v
        self.written_step[:P] = self.t + 1

    def step(self, x: np.ndarray, A: np.ndarray, keep_after=None, logit_rows=None):
        self.t += 1
        m = self.m
        A = np.asarray(A, dtype=np.int64)
        h = self.fw.embed(x[A])
        for l in range(m.n_layers):
            q, k, v = self.fw.qkv(l, h, A)
            self.K[l, A] = k
            self.V[l, A] = v
            h = self.fw.after_attention(l, h, attention(q, self.K[l], self.V[l]))
        self.written_step[A] = self.t
        return _scatter_logits(self.fw, h, A, logit_rows, self.L)


# ---------------------------------------------------------------------------
# confidence and selection
# ---------------------------------------------------------------------------

SCORE_MAXPROB, SCORE_MARGIN, SCORE_NEG_ENTROPY = 0, 1, 2


def confidence(logits_row: np.ndarray, mask_id: int, score: int = SCORE_MAXPROB) -> Tuple[float, int]:
    """Score of a position and its predicted token (argmax, lowest id on ties);
    the mask token itself is never predicted.  Sec. 3.1 names the remasking
    scores: the largest softmax probability (SCORE_MAXPROB, "most confident"),
    the margin between the two most probable values (SCORE_MARGIN), and, as
    the case studies label Dream's sampler, the entropy: SCORE_NEG_ENTROPY =
    sum_j p_j log p_j, so that a larger score again means more confident."""
    l = np.array(logits_row, dtype=np.float64)
    l[mask_id] = -np.inf
    pred = int(np.argmax(l))
    p = np.exp(l - l[pred])
    p = p / p.sum()
    if score == SCORE_MAXPROB:
        return float(p[pred]), pred
    if score == SCORE_MARGIN:
        rest = np.delete(p, pred)
        return float(p[pred] - rest.max()), pred
    if score == SCORE_NEG_ENTROPY:
        nz = p[p > 0]
        return float(np.sum(nz * np.log(nz))), pred
    raise ValueError("unknown score")


def select_unmask(conf: np.ndarray, masked: np.ndarray, cand_lo: int, cand_hi: int, k: int) -> List[int]:
    """k candidate positions (masked, inside [cand_lo, cand_hi)) with the
    largest confidence; ties go to the lower position; NaN counts as -inf.
    Returned in order of decreasing confidence."""
    cands = [i for i in range(cand_lo, cand_hi) if masked[i]]
    if len(cands) < k:
        raise ValueError("fewer than k candidates")
    def key(i):
        c = conf[i]
        c = -np.inf if np.isnan(c) else c
        return (-c, i)
    return sorted(cands, key=key)[:k]


# ---------------------------------------------------------------------------
# generation
# ---------------------------------------------------------------------------

@dataclasses.dataclass
class StepTrace:
    t: int
    refresh: bool
    x_in: np.ndarray          # tokens fed to step t
    masked_in: np.ndarray     # M_t
    active: np.ndarray        # A_t
    head_rows: np.ndarray     # H_t
    cand: Tuple[int, int]
    conf: np.ndarray          # [L], -inf outside H_t
    pred: np.ndarray          # [L], -1 outside H_t
    chosen: List[int]         # D_t
    written_step: np.ndarray  # [L] after the step
    logits: Optional[np.ndarray] = None   # [len(H_t), V] rows in H_t order
    prefilled: int = 0        # rows computed in a prompt-only pass before the step's own rows (isolated prefill)


class Sampler:
    """The sampling loop of one sequence, one step per call of ``step()``.
    order: [T, k] predefined positions (required for Greedy; optional replay
    for the other policies)."""

    def __init__(self, model: Model, W: Dict, prompt: np.ndarray, gen_len: int, k: int, pol: Policy,
                 block_len: Optional[int] = None, order: Optional[np.ndarray] = None, form: str = "literal",
                 rnd=_identity, keep_logits: bool = False, dtype=np.float64, all_logits: bool = False):
        self.model, self.pol, self.k, self.order, self.form = model, pol, k, order, form
        self.keep_logits, self.all_logits = keep_logits, all_logits
        self.P = len(prompt)
        self.L = self.P + gen_len
        self.T = gen_len // k
        assert gen_len % k == 0
        self.block_len = gen_len if block_len is None else block_len
        assert self.block_len % k == 0 and gen_len % self.block_len == 0
        self.x = np.concatenate([np.asarray(prompt, dtype=np.int64), np.full(gen_len, model.mask_id, dtype=np.int64)])
        self.M = np.zeros(self.L, dtype=np.uint8)
        self.M[self.P:] = 1
        self.cache = (LiteralCache(model, W, self.L, rnd) if form == "literal"
                      else SlotCache(model, W, self.L, rnd, dtype))
        self.M_prev, self.D_prev, self.t = None, None, 0
        if pol.kind == POLICY_GREEDY:
            assert order is not None, "Greedy needs a predefined decoding order"

    def step(self) -> StepTrace:
        self.t += 1
        t, pol, L, P, M, x = self.t, self.pol, self.L, self.P, self.M, self.x
        D_given = [int(p) for p in self.order[t - 1]] if self.order is not None else None
        A = active_set(t, pol, L, P, self.M_prev, M, D_given, self.D_prev)
        isolated = t == 1 and pol.isolated_prefill and P > 0
        if isolated:
            assert pol.kind in (POLICY_PREFILL, POLICY_PD), "isolated prefill belongs to the Prefill / PD policies"
            self.cache.prefill(x[:P])
            A = np.arange(P, L, dtype=np.int64)
        refresh = isolated or len(A) == L or (pol.kind == POLICY_PD and is_refresh_step(t, pol))
        blk = (t - 1) // (self.block_len // self.k)
        cand = (P + blk * self.block_len, P + (blk + 1) * self.block_len)
        if pol.kind == POLICY_GREEDY:
            H = np.array(sorted(D_given), dtype=np.int64)
        else:
            H = np.array([i for i in range(cand[0], cand[1]) if M[i]], dtype=np.int64)
        # Models adapted from autoregressive ones predict token j at row j-1 (Appendix B).  With the
        # unshifted caching rule the K/V of every position are cached exactly as before; the rows
        # j-1 of the candidates j are simply computed as well, because their outputs are needed.
        src = H - 1 if pol.shift else H
        if pol.shift == 2:
            # Un&Right-Shift: row j may be served from the cache only when the policy would cache both
            # position j (its input is fixed) and position j+1 (the token it predicts is decoded)
            left = A[A >= 1] - 1
            A = np.union1d(A, left).astype(np.int64)
        if pol.shift:
            assert len(H) == 0 or H.min() >= 1, "a shifted head cannot predict position 0"
            A = np.union1d(A, src).astype(np.int64)
        # what the next step will read from the cache, when already known (Algorithm 1's Reorder)
        keep_after = None
        if self.form == "literal" and pol.kind in (POLICY_DECODE, POLICY_PD) and pol.delay == 1:
            keep_after = [p for p in range(L) if not M[p]]      # next active set is M_t
        logits = self.cache.step(x, A, keep_after, None if self.all_logits else src)
        conf = np.full(L, -np.inf)
        pred = np.full(L, -1, dtype=np.int64)
        for i, si in zip(H, src):
            conf[i], pred[i] = confidence(logits[int(si)], self.model.mask_id, pol.score)
        chosen = D_given if D_given is not None else select_unmask(conf, M, cand[0], cand[1], self.k)
        st = StepTrace(t, refresh, x.copy(), M.copy(), A.copy(), H, cand, conf, pred, list(chosen),
                       self.cache.written_step.copy(), logits[src].copy() if self.keep_logits else None,
                       P if isolated else 0)
        self.M_prev = M.copy()
        for p in chosen:
            x[p] = pred[p]
            M[p] = 0
        self.D_prev = list(chosen)
        return st


def generate_one(model: Model, W: Dict, prompt: np.ndarray, gen_len: int, k: int, pol: Policy,
                 block_len: Optional[int] = None, order: Optional[np.ndarray] = None,
                 form: str = "literal", rnd=_identity, keep_logits: bool = False,
                 n_steps: Optional[int] = None, dtype=np.float64) -> List[StepTrace]:
    """Sampling loop of one sequence: T = gen_len / k steps (or n_steps)."""
    s = Sampler(model, W, prompt, gen_len, k, pol, block_len, order, form, rnd, keep_logits, dtype)
    return [s.step() for _ in range(n_steps or s.T)]


def final_tokens(trace: List[StepTrace]) -> np.ndarray:
    last = trace[-1]
    x = last.x_in.copy()
    for p in last.chosen:
        x[p] = last.pred[p]
    return x


def cache_ratio(trace: List[StepTrace]) -> float:
    """Mean over steps of the fraction of rows served from the cache."""
    L = len(trace[0].x_in)
    return float(np.mean([(L - len(s.active) - s.prefilled) / L for s in trace]))
