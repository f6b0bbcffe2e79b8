"""Runs the CUDA path and the CPU oracle side by side on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle.ptenc_oracle import OracleCache
from ptenc_inputs import SynthInputs

TOL_OUT = {"fp32": 1e-5, "bf16": 2e-2}   # max-abs on attention outputs (the stated targets)
TOL_LSE = {"fp32": 1e-5, "bf16": 1e-4}   # lse is fp32 on both storage types; bf16 inputs are exact in fp32
TOL_STATE = 1e-4                          # fp32 accumulation of the state vs float64, unit-norm rows


def np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().double().cpu().numpy()


class Pair:
    """A CUDA cache and an oracle cache with identical configuration and encoder parameters."""

    def __init__(self, pt, *, n_layers, batch, n_q_heads, n_kv_heads, head_dim, window, evict_chunk=1,
                 n_global=8, rank=8, dtype="bf16", normalize_mode=0, encode_enabled=1, seed=0,
                 kv_scale=1.0, set_encoder=True, global_kv=True, attn_consumer_warps=0):
        self.pt = pt
        self.shape = dict(n_layers=n_layers, batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                          head_dim=head_dim)
        self.L, self.B, self.Hq, self.Hkv, self.D = n_layers, batch, n_q_heads, n_kv_heads, head_dim
        self.W, self.E, self.dtype = window, evict_chunk, dtype
        self.gen = SynthInputs(seed=seed, dtype=dtype, n_global=n_global, rank=rank, kv_scale=kv_scale,
                               device="cuda:0", **self.shape)
        cfg = pt.make_config(window=window, evict_chunk=evict_chunk, n_global=n_global, rank=rank, dtype=dtype,
                             normalize_mode=normalize_mode, encode_enabled=encode_enabled,
                             attn_consumer_warps=attn_consumer_warps, **self.shape)
        self.cache = pt.Cache(cfg)
        if attn_consumer_warps and self.cache.info()["tensor_core_attn"]:
            assert self.cache.attn_launch_info(-1)["consumer_warps"] == attn_consumer_warps
        self.orc = OracleCache(window=window, evict_chunk=evict_chunk, n_global=n_global, rank=rank,
                               normalize_mode=normalize_mode, encode_enabled=encode_enabled, **self.shape)
        if set_encoder:
            for l in range(n_layers):
                P = self.gen.encoder_params(l)
                if not global_kv:
                    P["k_g"] = P["v_g"] = None
                self.cache.set_encoder(l, P["Wq_a"], P["Wk_a"], P["Wv_a"], P["q_g"], P["k_g"], P["v_g"])
                self.orc.set_encoder(l, **{k: (None if v is None else np64(v)) for k, v in P.items()})
        self.out = torch.zeros(n_layers, batch, n_q_heads, head_dim, dtype=self.cache.torch_dtype, device="cuda:0")
        self.out2 = torch.zeros_like(self.out)
        self.lse = torch.zeros(n_layers, batch, n_q_heads, dtype=torch.float32, device="cuda:0")

    def close(self):
        self.cache.close()

    def prefill(self, n_prompt, p_max, tensor_id=50):
        """Pins a synthetic prompt of n_prompt[b] tokens per sequence on both sides."""
        shape = (self.L, self.B, p_max, self.Hkv, self.D)
        Kp = self.gen.generic(tensor_id, 0, shape, 1.0)
        Vp = self.gen.generic(tensor_id + 1, 0, shape, 1.0)
        n_dev = torch.as_tensor(np.asarray(n_prompt), dtype=torch.int32, device="cuda:0")
        self.cache.prefill(-1, Kp, Vp, n_dev, p_max)
        for l in range(self.L):
            self.orc.prefill(l, np64(Kp[l]), np64(Vp[l]), n_prompt)

    def check_ring(self):
        for l in range(self.L):
            head, count, n_app = self.cache.get_ring(l)
            pinned = self.cache.get_pinned(l).cpu().numpy()
            oh, oc, on = self.orc.ring(l)
            count = count.cpu().numpy()
            assert np.array_equal(count, oc), (l, count, oc)
            assert np.array_equal(n_app.cpu().numpy(), on)
            assert np.array_equal(pinned, self.orc.pinned_count(l))
            live = oc > 0
            # the library counts the head from the first slot after the pinned entries
            assert np.array_equal((head.cpu().numpy() + pinned)[live], oh[live])

    def check_state(self, tol=TOL_STATE, rel=False):
        worst = 0.0
        for l in range(self.L):
            if self.orc.S[l] is None:
                continue
            S = np64(self.cache.get_state(l))
            ref = self.orc.S[l]
            err = np.abs(S - ref).max()
            if rel:
                err = err / max(1.0, np.abs(ref).max())
            worst = max(worst, err)
        assert worst <= tol, worst
        return worst

    def step(self, t, active=None, check=True, fused=True, all_layers=True):
        """One decode step on both sides.  Returns the max-abs output error over active sequences."""
        q = self.gen.step_q(t)
        k, v = self.gen.step_kv(t)
        act_dev = None if active is None else torch.as_tensor(active, dtype=torch.uint8, device="cuda:0")
        layers = [-1] if all_layers else list(range(self.L))
        for layer in layers:
            sl = slice(None) if layer == -1 else layer
            if fused:
                self.cache.decode_step(layer, q[sl], k[sl], v[sl], self.out[sl], act_dev)
            else:
                self.cache.append_evict(layer, k[sl], v[sl], act_dev)
                self.cache.encode(layer)
                self.cache.decode_attn(layer, q[sl], self.out[sl], act_dev)
        if check:
            # the attention alone once more on the same cache (it changes nothing): same outputs, plus the fp32
            # log-sum-exp, which is far more sensitive to a mis-counted tile than the rounded outputs are
            self.out2.zero_()
            self.lse.zero_()
            for layer in layers:
                sl = slice(None) if layer == -1 else layer
                self.cache.decode_attn(layer, q[sl], self.out2[sl], act_dev, self.lse[sl])
        worst = worst_lse = 0.0
        qn, kn, vn = np64(q), np64(k), np64(v)
        outn = np64(self.out)
        lsen = np64(self.lse)
        for l in range(self.L):
            o_ref, lse_ref, rec = self.orc.decode_step(l, qn[l], kn[l], vn[l], active)
            if check:
                m = np.ones(self.B, bool) if active is None else np.asarray(active, bool)
                m = m & ((self.orc.ring(l)[1] + self.orc.pinned_count(l)) > 0)
                if m.any():
                    worst = max(worst, np.abs(outn[l][m] - o_ref[m]).max())
                    worst_lse = max(worst_lse, np.abs(lsen[l][m] - lse_ref[m]).max())
        if check:
            assert worst <= TOL_OUT[self.dtype], (t, worst)
            assert worst_lse <= TOL_LSE[self.dtype], (t, worst_lse)
            ma = slice(None) if active is None else torch.as_tensor(np.asarray(active, bool), device="cuda:0")
            assert torch.equal(self.out[:, ma], self.out2[:, ma]), t
        return worst
