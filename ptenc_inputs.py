"""Seeded synthetic inputs for the Progressive Thought Encoding decode path.

This module is shared by the CPU oracle's tests and by the CUDA path's tests and
benchmark.  It contains none of the method's arithmetic: it only produces the
tensors the method consumes (queries, keys, values, encoder parameters, ragged
lengths), as a pure function of (seed, tensor id, step, element index), so any
element can be regenerated in isolation (random access) and the result is
bit-identical on CPU and on a CUDA device.

Recipe
------
A 32-bit integer hash of the element's counter picks one of 65536 equally likely
standard-normal quantiles z_i = Phi^-1((i + 1/2) / 65536).  The quantile table is
computed once on the host in float64, scaled, rounded to the storage dtype and
only then moved to the target device; generation is integer arithmetic plus one
gather, so no floating-point operation runs on the device.

The workloads this stands in for are the paper's rollouts (Sec. 4.1, "Models" and
"Implementation Details"): per decode step every layer receives one query vector
per query head and one key/value vector per KV head for every sequence.
"""
from __future__ import annotations

import numpy as np
import torch

_M32 = 0xFFFFFFFF
_MUL = 0x045D9F3B  # < 2**27, so a 32-bit value times it stays below 2**63

# tensor ids (part of the counter)
T_Q, T_K, T_V = 1, 2, 3
T_WQ, T_WK, T_WV, T_QG, T_KG, T_VG = 10, 11, 12, 13, 14, 15
T_LEN, T_ACTIVE = 20, 21
T_LORA_A, T_LORA_B, T_X = 30, 31, 32

_TABLE64 = None


def _quantile_table() -> np.ndarray:
    global _TABLE64
    if _TABLE64 is None:
        from scipy.special import ndtri
        p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        _TABLE64 = ndtri(p)
    return _TABLE64


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """32-bit avalanche hash on int64 tensors holding values in [0, 2**32)."""
    x = ((x >> 16) ^ x) * _MUL & _M32
    x = ((x >> 16) ^ x) * _MUL & _M32
    x = (x >> 16) ^ x
    return x


def _mix32_int(x: int) -> int:
    x &= _M32
    x = (((x >> 16) ^ x) * _MUL) & _M32
    x = (((x >> 16) ^ x) * _MUL) & _M32
    x = (x >> 16) ^ x
    return x & _M32


def _key(seed: int, tensor_id: int, step) -> "int | torch.Tensor":
    """Stream key for (seed, tensor, step).  `step` may be an int or an int64 tensor."""
    base = _mix32_int(_mix32_int(seed * 0x9E37 + 0x7F4A7C15) ^ (tensor_id * 0x85EBCA6B & _M32))
    if isinstance(step, torch.Tensor):
        return _mix32((step & _M32) ^ base)
    return _mix32_int((int(step) & _M32) ^ base)


def _storage(dtype: str) -> torch.dtype:
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[dtype]


class SynthInputs:
    """Random-access generator of one decode workload.

    Shapes follow the decode step: per step `q [L,B,Hq,D]`, `k,v [L,B,Hkv,D]`.
    `kv_scale` multiplies keys and values (0.5 for the 3B-shaped workload).
    """

    def __init__(self, *, seed: int, n_layers: int, batch: int, n_q_heads: int,
                 n_kv_heads: int, head_dim: int, dtype: str = "bf16",
                 kv_scale: float = 1.0, q_scale: float = 1.0,
                 n_global: int = 32, rank: int = 32, device="cpu"):
        self.seed, self.L, self.B = int(seed), n_layers, batch
        self.Hq, self.Hkv, self.D = n_q_heads, n_kv_heads, head_dim
        self.G, self.r = n_global, rank
        self.dtype = dtype
        self.kv_scale, self.q_scale = float(kv_scale), float(q_scale)
        self.device = torch.device(device)
        self._tables = {}

    # -- tables -----------------------------------------------------------------
    def _table(self, scale: float, device=None) -> torch.Tensor:
        device = self.device if device is None else torch.device(device)
        k = (float(scale), str(device))
        if k not in self._tables:
            t = torch.from_numpy(_quantile_table() * float(scale)).to(torch.float32)
            t = t.to(_storage(self.dtype))  # rounded on the host, then moved
            self._tables[k] = t.to(device)
        return self._tables[k]

    def _draw(self, key, idx: torch.Tensor, scale: float, device=None) -> torch.Tensor:
        h = _mix32((idx ^ key) & _M32)
        h = _mix32(h + 0x632BE5AB & _M32)
        return self._table(scale, device)[h & 0xFFFF]

    # -- per-step activations ------------------------------------------------------
    def _flat(self, H: int, device) -> torch.Tensor:
        n = self.L * self.B * H * self.D
        return torch.arange(n, dtype=torch.int64, device=device)

    def step_q(self, step: int, device=None) -> torch.Tensor:
        """Queries of decode step `step`: [L, B, Hq, D]."""
        device = self.device if device is None else torch.device(device)
        x = self._draw(_key(self.seed, T_Q, step), self._flat(self.Hq, device), self.q_scale, device)
        return x.view(self.L, self.B, self.Hq, self.D)

    def step_kv(self, step: int, device=None):
        """Keys and values of the token arriving at `step`: two [L, B, Hkv, D]."""
        device = self.device if device is None else torch.device(device)
        idx = self._flat(self.Hkv, device)
        k = self._draw(_key(self.seed, T_K, step), idx, self.kv_scale, device)
        v = self._draw(_key(self.seed, T_V, step), idx, self.kv_scale, device)
        shp = (self.L, self.B, self.Hkv, self.D)
        return k.view(shp), v.view(shp)

    # -- random access (one layer, one sequence) ------------------------------------
    def _idx_lb(self, layer: int, seq: int, H: int) -> torch.Tensor:
        base = (layer * self.B + seq) * H * self.D
        return torch.arange(H * self.D, dtype=torch.int64) + base

    def token_q(self, layer: int, seq: int, step: int) -> torch.Tensor:
        """[Hq, D] query of (layer, seq) at `step`, on the CPU."""
        x = self._draw(_key(self.seed, T_Q, step), self._idx_lb(layer, seq, self.Hq), self.q_scale, "cpu")
        return x.view(self.Hq, self.D)

    def token_kv(self, layer: int, seq: int, steps):
        """Keys/values of (layer, seq) for the given steps, on the CPU: two [n, Hkv, D]."""
        steps = torch.as_tensor(steps, dtype=torch.int64).view(-1, 1)
        idx = self._idx_lb(layer, seq, self.Hkv).view(1, -1)
        k = self._draw(_key(self.seed, T_K, steps), idx, self.kv_scale, "cpu")
        v = self._draw(_key(self.seed, T_V, steps), idx, self.kv_scale, "cpu")
        n = steps.shape[0]
        return k.view(n, self.Hkv, self.D), v.view(n, self.Hkv, self.D)

    # -- encoder parameters (Sec. 3.3): W^a_Q, W^a_K, W^a_V, q_g, k_g, v_g ----------------
    def encoder_params(self, layer: int, device=None):
        """Returns dict of tensors in the storage dtype.

        Scales keep the rows of one evicted token's contribution O(1):
        W^a_Q [r,d_q] ~ N(0,1/d_q), W^a_K [r,d_kv] ~ N(0,1/d_kv),
        W^a_V [r,d_kv] ~ N(0,1/(d_kv r)), q_g [G,d_q] ~ N(0,1/r), k_g,v_g [G,d_kv] ~ N(0,1).
        """
        device = self.device if device is None else torch.device(device)
        d_q, d_kv, G, r = self.Hq * self.D, self.Hkv * self.D, self.G, self.r
        spec = {
            "Wq_a": (T_WQ, (r, d_q), d_q ** -0.5),
            "Wk_a": (T_WK, (r, d_kv), d_kv ** -0.5),
            "Wv_a": (T_WV, (r, d_kv), (d_kv * r) ** -0.5),
            "q_g": (T_QG, (G, d_q), r ** -0.5),
            "k_g": (T_KG, (G, d_kv), self.kv_scale),
            "v_g": (T_VG, (G, d_kv), self.kv_scale),
        }
        out = {}
        for name, (tid, shape, scale) in spec.items():
            n = shape[0] * shape[1]
            idx = torch.arange(n, dtype=torch.int64, device=device)
            out[name] = self._draw(_key(self.seed, tid, layer), idx, scale, device).view(shape)
        return out

    # -- ragged lengths / activity ---------------------------------------------------------
    def lengths(self, lo: int, hi: int) -> torch.Tensor:
        """Per-sequence rollout lengths, uniform on {lo..hi}: int64 [B] on the CPU."""
        idx = torch.arange(self.B, dtype=torch.int64)
        h = _mix32((idx ^ _key(self.seed, T_LEN, 0)) & _M32)
        h = _mix32(h + 0x632BE5AB & _M32)
        return lo + h % (hi - lo + 1)

    def generic(self, tensor_id: int, stream: int, shape, scale: float, device=None) -> torch.Tensor:
        """Any other N(0, scale^2) tensor (e.g. LoRA maps), storage dtype."""
        device = self.device if device is None else torch.device(device)
        n = int(np.prod(shape))
        idx = torch.arange(n, dtype=torch.int64, device=device)
        return self._draw(_key(self.seed, tensor_id, stream), idx, scale, device).view(*shape)


# Workload shapes (batch, heads, window, rollout length) of the five configurations.
CONFIGS = {
    "tiny": dict(n_layers=1, batch=2, n_q_heads=4, n_kv_heads=1, head_dim=64, window=64,
                 n_global=16, rank=16, dtype="fp32", steps=256, kv_scale=1.0),
    "qwen3b": dict(n_layers=36, batch=64, n_q_heads=16, n_kv_heads=2, head_dim=128, window=1024,
                   n_global=32, rank=32, dtype="bf16", steps=4096, kv_scale=0.5),
    "qwen7b": dict(n_layers=28, batch=128, n_q_heads=28, n_kv_heads=4, head_dim=128, window=2048,
                   n_global=32, rank=32, dtype="bf16", steps=8192, kv_scale=1.0),
    "llama8b": dict(n_layers=32, batch=64, n_q_heads=32, n_kv_heads=8, head_dim=128, window=4096,
                    n_global=32, rank=32, dtype="bf16", steps=16384, kv_scale=1.0,
                    ragged=(2048, 16384)),
}


def stress_config(window: int, batch: int) -> dict:
    c = dict(CONFIGS["qwen7b"])
    c.update(window=window, batch=batch, steps=32768)
    return c


def make_inputs(cfg: dict, seed: int = 0, device="cpu") -> SynthInputs:
    return SynthInputs(seed=seed, n_layers=cfg["n_layers"], batch=cfg["batch"],
                       n_q_heads=cfg["n_q_heads"], n_kv_heads=cfg["n_kv_heads"],
                       head_dim=cfg["head_dim"], dtype=cfg["dtype"], kv_scale=cfg.get("kv_scale", 1.0),
                       n_global=cfg["n_global"], rank=cfg["rank"], device=device)
