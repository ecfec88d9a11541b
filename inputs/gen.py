"""Counter-based seeded tensors, identical bit for bit on CPU and CUDA.

Every value is a pure function of (seed, tensor name, element index):

    s   = key + (index + 1) * 0x9E3779B97F4A7C15          (mod 2^64)
    h   = splitmix64 finaliser of s
    k   = top 32 bits of h
    z   = T[k >> 16] + D[k >> 16] * ((k & 0xffff) / 65536)

where T is a 65537-knot table of standard-normal quantiles (computed once on the
CPU in float64, stored as float32, D its first differences), so z is a
piecewise-linear inverse-CDF sample of N(0, 1) clipped at about +-4.3 sigma.
Only integer ops, table lookups and separately rounded float32 multiply / add
are used, so a tensor generated on the GPU equals the one generated on the CPU.
Nothing here belongs to the decoding method itself.
"""
from __future__ import annotations

import math
from typing import Dict, Iterable, List, Tuple

import torch

from .configs import ModelShape

_GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_CHUNK = 1 << 24


def _s64(c: int) -> int:
    c &= (1 << 64) - 1
    return c - (1 << 64) if c >= (1 << 63) else c


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix_py(z: int) -> int:
    z &= (1 << 64) - 1
    z = ((z ^ (z >> 30)) * _M1) & ((1 << 64) - 1)
    z = ((z ^ (z >> 27)) * _M2) & ((1 << 64) - 1)
    return z ^ (z >> 31)


def _name_key(seed: int, name: str) -> int:
    h = 0xCBF29CE484222325                       # FNV-1a over the name
    for b in name.encode():
        h = ((h ^ b) * 0x100000001B3) & ((1 << 64) - 1)
    return _mix_py(_mix_py(seed + _GOLD) ^ h)


def _hash(idx: torch.Tensor, key: int) -> torch.Tensor:
    z = (idx + 1) * _s64(_GOLD) + _s64(key)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


_tables: Dict[str, Tuple[torch.Tensor, torch.Tensor]] = {}


def _normal_tables(device) -> Tuple[torch.Tensor, torch.Tensor]:
    dev = str(torch.device(device))
    if "cpu" not in _tables:
        j = torch.arange(65537, dtype=torch.float64)
        p = (j + 0.5) / 65537.0
        t = (math.sqrt(2.0) * torch.erfinv(2.0 * p - 1.0)).to(torch.float32)
        _tables["cpu"] = (t, (t[1:] - t[:-1]).contiguous())
    if dev not in _tables:
        t, d = _tables["cpu"]
        _tables[dev] = (t.to(device), d.to(device))
    return _tables[dev]


def normal_tensor(shape: Iterable[int], std: float, seed: int, name: str,
                  dtype=torch.float32, device="cpu") -> torch.Tensor:
    """N(0, std) tensor (quantile-table normal, see the module docstring)."""
    shape = tuple(int(s) for s in shape)
    n = 1
    for s in shape:
        n *= s
    key = _name_key(seed, name)
    T, D = _normal_tables(device)
    out = torch.empty(n, dtype=dtype, device=device)
    std32 = torch.tensor(std, dtype=torch.float32, device=device)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        k = _lsr(_hash(idx, key), 32)
        i = k >> 16
        frac = (k & 0xFFFF).to(torch.float32) * (1.0 / 65536.0)
        z = D[i] * frac
        z = z + T[i]
        z = z * std32
        out[lo:hi] = z.to(dtype)
    return out.view(shape)


def uniform_ids(n: int, high: int, seed: int, name: str, device="cpu") -> torch.Tensor:
    """n integer ids uniform on [0, high) as int32."""
    idx = torch.arange(n, dtype=torch.int64, device=device)
    k = _lsr(_hash(idx, _name_key(seed, name)), 32)
    return (k % high).to(torch.int32)


def uniform_floats(n: int, seed: int, name: str) -> List[float]:
    """n Python floats uniform on [0, 1) (CPU only; used by the tree recipe)."""
    idx = torch.arange(n, dtype=torch.int64)
    k = _lsr(_hash(idx, _name_key(seed, name)), 32)
    return (k.to(torch.float64) / 4294967296.0).tolist()


def _layer_specs(prefix: str, d: int, f: int) -> List[Tuple[str, Tuple[int, ...], str]]:
    return [
        (prefix + "attn_norm", (d,), "ones"),
        (prefix + "wq", (d, d), "normal"),
        (prefix + "wk", (d, d), "normal"),
        (prefix + "wv", (d, d), "normal"),
        (prefix + "wo", (d, d), "normal"),
        (prefix + "ffn_norm", (d,), "ones"),
        (prefix + "w_gate", (f, d), "normal"),
        (prefix + "w_up", (f, d), "normal"),
        (prefix + "w_down", (d, f), "normal"),
    ]


def weight_specs(shape: ModelShape) -> List[Tuple[str, Tuple[int, ...], str]]:
    """(name, shape, init) for every tensor of the target and the draft module.

    All linear weights are stored [out_features, in_features] row-major.
    """
    d, f, v, K = shape.d_model, shape.d_ffn, shape.vocab, shape.K
    specs: List[Tuple[str, Tuple[int, ...], str]] = [("tok_emb", (v, d), "normal")]
    for i in range(shape.n_layers):
        specs += _layer_specs(f"layers.{i}.", d, f)
    specs += [("final_norm", (d,), "ones"), ("lm_head", (v, d), "normal")]
    for s in range(1, shape.n_sal + 1):
        specs.append((f"draft.fc{s}", (d, 2 * d if shape.use_sampled_token else d), "normal"))
        specs += _layer_specs(f"draft.sal{s}.", d, f)
    for k in range(K):
        specs.append((f"draft.mlp.{k}.w", (d, d), "normal"))
        specs.append((f"draft.mlp.{k}.b", (d,), "normal"))
    specs.append(("draft.pe", (K, d), "normal"))
    for l in range(shape.aeb_layers):
        for w in ("wq", "wk", "wv", "wo"):
            specs.append((f"draft.aeb.{l}.{w}", (d, d), "normal"))
    for k in range(K):
        if shape.lm_rank > 0:                      # two low-rank factors instead of the [V, d] matrix
            specs.append((f"draft.lm_head.{k}.a", (shape.lm_rank, d), "normal"))
            specs.append((f"draft.lm_head.{k}.b", (v, shape.lm_rank), "normal"))
        else:
            specs.append((f"draft.lm_head.{k}", (v, d), "normal"))
    return specs


def tensor_std(name: str, shp: Tuple[int, ...], std: float, init: str) -> float:
    """Standard deviation of one tensor.  init "normal": `std` for every tensor (the benchmark's N(0, 0.02)).
    init "fan_in": every linear map gets 1 / sqrt(in_features), so that it neither amplifies nor damps its
    input whatever the width (embedding rows have unit variance; biases and position embeddings 0.5)."""
    if init == "normal":
        return std
    if name == "tok_emb":
        return 1.0
    if len(shp) == 1 or name == "draft.pe":
        return 0.5
    return 1.0 / math.sqrt(shp[-1])


def make_weights(shape: ModelShape, seed: int = 0, device="cpu", std: float = 0.02,
                 only=None, init: str = "normal") -> Dict[str, torch.Tensor]:
    """All weights of `shape` in its storage dtype; norm gains 1; the rest normal (see tensor_std)."""
    assert init in ("normal", "fan_in")
    dtype = torch.float32 if shape.dtype == "fp32" else torch.bfloat16
    out: Dict[str, torch.Tensor] = {}
    for name, shp, kind in weight_specs(shape):
        if only is not None and not only(name):
            continue
        if kind == "ones":
            out[name] = torch.ones(shp, dtype=dtype, device=device)
        else:
            out[name] = normal_tensor(shp, tensor_std(name, shp, std, init), seed, name, dtype=dtype, device=device)
    return out


def make_prompt(shape: ModelShape, seed: int = 1, n: int = 0, device="cpu") -> torch.Tensor:
    n = n or shape.prompt_len
    return uniform_ids(n, shape.vocab, seed, "prompt", device=device)
