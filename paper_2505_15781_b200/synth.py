"""Seeded synthetic inputs: weights, prompts, decoding orders, active-index sets.

This module holds no arithmetic of the method.  It only makes reproducible
numbers.  Both the CPU oracle's tests and the CUDA path are fed from here, so
that the two sides see identical data without sharing any code of the method.

Weights come from a counter-based generator: element ``i`` of tensor
``(seed, layer, tensor_id)`` is ``table[hash32(i, key) >> 16] * std`` where
``table`` holds the 65536 mid-point quantiles of the standard normal
distribution.  Everything before the table lookup is integer arithmetic, so
the CPU (numpy or torch) and the GPU (torch) produce bit-identical tensors and
an 8-billion-parameter model can be filled on the device in a few seconds.
The result is N(0, std) quantised to 16-bit quantiles (sample std 0.99996*std).
"""
from __future__ import annotations

import dataclasses
import functools
from typing import Dict, List, Optional, Sequence

import numpy as np

_M32 = 0xFFFFFFFF
_C1 = 0x7FEB352D
_C2 = 0x846CA68B

# tensor ids inside one layer / global tensors
TENSOR_IDS = {
    "attn_norm": 0, "wq": 1, "wk": 2, "wv": 3, "wo": 4,
    "ffn_norm": 5, "wg": 6, "wu": 7, "wd": 8,
    "embed": 100, "final_norm": 101, "head": 102,
}


@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Shape of a bidirectional pre-norm decoder (RMSNorm, RoPE, SwiGLU)."""
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

    @property
    def d_q(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim

    def params_per_layer(self) -> int:
        d = self.d_model
        return d * self.d_q + 2 * d * self.d_kv + self.d_q * d + 3 * d * self.d_ffn

    def with_layers(self, n: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n)


def tiny_shape() -> ModelShape:
    return ModelShape(2, 256, 4, 4, 64, 688, 1024, 1023)


def llada_shape(n_layers: int = 32) -> ModelShape:
    return ModelShape(n_layers, 4096, 32, 32, 128, 12288, 126464, 126463)


def dream_shape(n_layers: int = 28) -> ModelShape:
    return ModelShape(n_layers, 3584, 28, 4, 128, 18944, 152064, 152063)


# ---------------------------------------------------------------------------
# counter-based generator
# ---------------------------------------------------------------------------

@functools.lru_cache(maxsize=None)
def quantile_table() -> np.ndarray:
    """65536 mid-point quantiles of N(0,1) as float32."""
    from scipy.special import ndtri
    u = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
    return ndtri(u).astype(np.float32)


def _splitmix64(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    return z ^ (z >> 31)


def tensor_key(seed: int, layer: int, tensor_id: int) -> (int, int):
    """Two 32-bit keys for one tensor (layer = -1 for global tensors)."""
    z = _splitmix64(_splitmix64(seed & _M32) ^ ((layer + 1) << 20) ^ tensor_id)
    return z & _M32, (z >> 32) & _M32


def _np_mul32(x: np.ndarray, c: int) -> np.ndarray:
    return (x * np.uint64(c)) & np.uint64(_M32)


def _np_hash32(x: np.ndarray) -> np.ndarray:
    x = x ^ (x >> np.uint64(16))
    x = _np_mul32(x, _C1)
    x = x ^ (x >> np.uint64(15))
    x = _np_mul32(x, _C2)
    x = x ^ (x >> np.uint64(16))
    return x


def hash_u16_numpy(start: int, n: int, k1: int, k2: int) -> np.ndarray:
    """Plain numpy form of the generator (used for small tensors and as the
    cross-check of the torch form)."""
    i = np.arange(start, start + n, dtype=np.uint64)
    x = _np_hash32((i ^ np.uint64(k1)) & np.uint64(_M32))
    x = _np_hash32((x + np.uint64(k2)) & np.uint64(_M32))
    return (x >> np.uint64(16)).astype(np.int64)


def _t_mul32(x, c: int):
    # (x * c) mod 2^32 for 0 <= x < 2^32 held in int64, without ever
    # overflowing int64: split x into 16-bit halves.
    lo = (x & 0xFFFF) * c
    hi = (((x >> 16) * c) & 0xFFFF) << 16
    return (lo + hi) & _M32


def _t_hash32(x):
    x = x ^ (x >> 16)
    x = _t_mul32(x, _C1)
    x = x ^ (x >> 15)
    x = _t_mul32(x, _C2)
    x = x ^ (x >> 16)
    return x


def hash_u16_torch(start: int, n: int, k1: int, k2: int, device):
    import torch
    i = torch.arange(start, start + n, dtype=torch.int64, device=device)
    x = _t_hash32((i ^ k1) & _M32)
    x = _t_hash32((x + k2) & _M32)
    return x >> 16


def normal_tensor(seed: int, layer: int, name: str, shape: Sequence[int], std: float,
                  dtype="float32", device="cpu", chunk: int = 1 << 26):
    """Tensor of N(0,std) quantile values, as torch tensor of ``dtype``
    ('float32' or 'bfloat16', the latter rounded to nearest-even from fp32)."""
    import torch
    k1, k2 = tensor_key(seed, layer, TENSOR_IDS[name])
    n = int(np.prod(shape))
    tdtype = {"float32": torch.float32, "bfloat16": torch.bfloat16}[dtype]
    table = torch.from_numpy(quantile_table()).to(device)
    out = torch.empty(n, dtype=tdtype, device=device)
    stdt = torch.tensor(std, dtype=torch.float32, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        u = hash_u16_torch(s, m, k1, k2, device)
        out[s:s + m] = (table[u] * stdt).to(tdtype)
    return out.view(*shape)


def normal_tensor_numpy(seed: int, layer: int, name: str, shape: Sequence[int], std: float) -> np.ndarray:
    k1, k2 = tensor_key(seed, layer, TENSOR_IDS[name])
    n = int(np.prod(shape))
    u = hash_u16_numpy(0, n, k1, k2)
    return (quantile_table()[u] * np.float32(std)).reshape(shape)


def layer_tensor_shapes(ms: ModelShape) -> Dict[str, tuple]:
    """Weight matrices are stored [out_features, in_features] row-major."""
    d, f = ms.d_model, ms.d_ffn
    return {
        "wq": (ms.d_q, d), "wk": (ms.d_kv, d), "wv": (ms.d_kv, d), "wo": (d, ms.d_q),
        "wg": (f, d), "wu": (f, d), "wd": (d, f),
    }


def norm_gain(seed: int, layer: int, name: str, d: int, device="cpu", spread: float = 0.1):
    """Gain vector of one RMSNorm: 1 + spread * N(0,1) from the same counter-based generator (fp32).
    Every norm of a model gets its own values, so a gain that is dropped, or taken from the wrong
    norm, changes the logits."""
    return normal_tensor(seed, layer, name, (d,), spread, "float32", device) + 1.0


def make_weights(ms: ModelShape, seed: int = 0, dtype: str = "float32", device="cpu",
                 std: float = 0.02) -> Dict[str, object]:
    """All tensors of a model: {'embed','final_norm','head', 'layers':[{...}]}.
    Matrices are N(0,std) in ``dtype``; norm gains are 1 + 0.1 * N(0,1) (fp32)."""
    w: Dict[str, object] = {}
    w["embed"] = normal_tensor(seed, -1, "embed", (ms.vocab, ms.d_model), std, dtype, device)
    w["head"] = normal_tensor(seed, -1, "head", (ms.vocab, ms.d_model), std, dtype, device)
    w["final_norm"] = norm_gain(seed, -1, "final_norm", ms.d_model, device)
    layers: List[Dict[str, object]] = []
    for l in range(ms.n_layers):
        lw = {}
        for name, shp in layer_tensor_shapes(ms).items():
            lw[name] = normal_tensor(seed, l, name, shp, std, dtype, device)
        lw["attn_norm"] = norm_gain(seed, l, "attn_norm", ms.d_model, device)
        lw["ffn_norm"] = norm_gain(seed, l, "ffn_norm", ms.d_model, device)
        layers.append(lw)
    w["layers"] = layers
    return w


def weights_to_numpy(w: Dict[str, object], dtype=np.float64) -> Dict[str, object]:
    """Same values as plain numpy arrays (bf16 values are exactly representable)."""
    def cv(t):
        return t.detach().to("cpu").float().numpy().astype(dtype)
    out = {k: cv(v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: cv(v) for k, v in lw.items()} for lw in w["layers"]]
    return out


# ---------------------------------------------------------------------------
# token-level inputs
# ---------------------------------------------------------------------------

def make_prompt(batch: int, prompt_len: int, hi: int, seed: int = 0) -> np.ndarray:
    """Prompt ids uniform in [0, hi) as int32 [batch, prompt_len]."""
    rng = np.random.Generator(np.random.PCG64(seed + 1000))
    return rng.integers(0, hi, size=(batch, prompt_len), dtype=np.int64).astype(np.int32)


def initial_state(prompt: np.ndarray, gen_len: int, mask_id: int):
    """x_1 = [prompt ; mask_id * gen_len], M_1 = generation region."""
    b, p = prompt.shape
    x = np.full((b, p + gen_len), mask_id, dtype=np.int32)
    x[:, :p] = prompt
    m = np.zeros((b, p + gen_len), dtype=np.uint8)
    m[:, p:] = 1
    return x, m


def random_order(batch: int, prompt_len: int, gen_len: int, k: int, seed: int = 0) -> np.ndarray:
    """A predefined decoding order: int32 [T, batch, k] of positions, a seeded
    permutation of the generation region per sequence."""
    rng = np.random.Generator(np.random.PCG64(seed + 2000))
    t = gen_len // k
    out = np.empty((t, batch, k), dtype=np.int32)
    for b in range(batch):
        perm = rng.permutation(gen_len).astype(np.int32) + prompt_len
        out[:, b, :] = perm.reshape(t, k)
    return out


def random_active_set(seq_len: int, n_active: int, seed: int = 0) -> np.ndarray:
    """Ascending int32 indices of n_active rows drawn uniformly without replacement."""
    rng = np.random.Generator(np.random.PCG64(seed + 3000))
    return np.sort(rng.choice(seq_len, size=n_active, replace=False)).astype(np.int32)


def random_mask_state(batch: int, prompt_len: int, gen_len: int, n_unmasked: int, hi: int, seed: int = 0):
    """A mid-generation state: prompt + generation region where n_unmasked
    random positions per sequence are already decoded (random ids)."""
    rng = np.random.Generator(np.random.PCG64(seed + 4000))
    x, m = initial_state(make_prompt(batch, prompt_len, hi, seed), gen_len, hi)
    for b in range(batch):
        pos = rng.choice(gen_len, size=n_unmasked, replace=False) + prompt_len
        x[b, pos] = rng.integers(0, hi, size=n_unmasked)
        m[b, pos] = 0
    return x, m
