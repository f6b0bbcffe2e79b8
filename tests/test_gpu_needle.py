"""Decode attention with a dominant key per unit ("needle"): a test that a mis-counted tile cannot pass.

With N(0,1) activations and windows of thousands of tokens every softmax weight is tiny, so a K/V tile that the
kernel dropped or counted twice moves the rounded outputs by less than the output tolerance.  Here every
(layer, sequence, KV head) unit gets queries that are multiples of ONE of its cached keys, so that this key's logit
towers over the rest (Sec. 3.1: the softmax then puts all weight on it): the output must be that token's value row
and the log-sum-exp must be that logit.  A dropped tile gives some other row (error of order 1); a tile counted
twice leaves the output alone but raises the log-sum-exp by log 2.  From launch to launch the needle of each unit
moves on by one tile, so every unit is tested at every tile position: the first tile, the last, the tile that holds
the wrap of the ring, partially filled tiles, and every tile at which the persistent schedule splits a unit between
two CTAs.

Two checks per launch: every unit against the value row and the key norm read back from the rings (a property that
holds at any size), and a few sampled units against the float64 oracle, whose inputs (the unit's keys, values and the
needle query) are regenerated from the seeded generator and never read from the device.
"""
import numpy as np
import pytest
import torch

import paper_2602_16839_b200 as pt
from oracle.ptenc_oracle import attention_gqa
from ptenc_inputs import CONFIGS, make_inputs

from _harness import TOL_LSE, TOL_OUT, np64

pytestmark = pytest.mark.gpu


def _ring_views(cache, L, B, Hkv, W, D):
    base = cache.workspace.data_ptr()
    views = []
    for region in (pt.binding.REGION_K, pt.binding.REGION_V):
        ptr, n = cache.workspace_region(region)
        assert n == L * B * Hkv * W * D * 2
        views.append(cache.workspace[ptr - base: ptr - base + n].view(torch.bfloat16).view(L, B, Hkv, W, D))
    return views


def _run_needles(c, L, T_list, warps, n_launches=None, n_sampled=5, seed=0):
    """Fills the rings with T tokens (each T of T_list in turn, continuing the same rollout), then runs one attention
    launch per tile position with a needle in every unit."""
    B, Hq, Hkv, D, W = c["batch"], c["n_q_heads"], c["n_kv_heads"], c["head_dim"], c["window"]
    g = Hq // Hkv
    dev = "cuda:0"
    torch.cuda.empty_cache()
    gen = make_inputs({**c, "n_layers": L}, seed=seed, device=dev)
    cfg = pt.make_config(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W, dtype="bf16",
                         attn_consumer_warps=warps)
    cache = pt.Cache(cfg)
    info = cache.attn_launch_info(-1)
    tile = info["tile_tokens"]
    Kr, Vr = _ring_views(cache, L, B, Hkv, W, D)
    rng = np.random.default_rng(7 + seed)
    # sampled units for the oracle: first and last unit of the launch and a few in between
    units = {(0, 0, 0), (L - 1, B - 1, Hkv - 1)}
    while len(units) < n_sampled:
        units.add((int(rng.integers(L)), int(rng.integers(B)), int(rng.integers(Hkv))))
    units = sorted(units)
    # query of head a = the needle's key scaled so that its own logit is 28 + a whatever the key's norm; the other
    # tokens' logits are then N(0, ~3^2) and hold less than 1e-5 of the softmax mass even at 4096 tokens
    peak = torch.tensor([28.0 + a for a in range(g)], dtype=torch.float32, device=dev)
    li = torch.arange(L, device=dev)[:, None, None].expand(L, B, Hkv)
    bi = torch.arange(B, device=dev)[None, :, None].expand(L, B, Hkv)
    hi = torch.arange(Hkv, device=dev)[None, None, :].expand(L, B, Hkv)
    out = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device=dev)
    lse = torch.zeros(L, B, Hq, dtype=torch.float32, device=dev)
    t_done = 0
    worst_out = worst_lse = worst_all_out = worst_all_lse = 0.0
    n_oracle = 0
    for T in T_list:
        for t in range(t_done, T):
            k, v = gen.step_kv(t)
            cache.append_evict(-1, k, v)
        t_done = T
        n_live = min(T, W)
        n_tiles = (n_live + tile - 1) // tile
        # slot -> token index for a FIFO ring after T arrivals: the newest token with t = slot (mod W)
        tok_of_slot = lambda s: s + ((T - 1 - s) // W) * W
        unit_cache = {}
        for u in units:                                   # the unit's live keys/values, regenerated once
            l, b, h = u
            toks = [tok_of_slot(s) for s in range(n_live)]
            Ku, Vu = gen.token_kv(l, b, toks)
            unit_cache[u] = (np64(Ku[:, h]), np64(Vu[:, h]))
        offs = torch.as_tensor(rng.integers(0, n_tiles, (L, B, Hkv)), device=dev)
        launches = range(n_tiles) if n_launches is None else range(n_launches)
        for i in launches:
            within = torch.as_tensor(rng.integers(0, tile, (L, B, Hkv)), device=dev)
            slot = ((offs + i) % n_tiles) * tile + within
            slot = torch.minimum(slot, torch.full_like(slot, n_live - 1))       # the last tile may be partial
            k_sel = Kr[li, bi, hi, slot].float()                                 # [L, B, Hkv, D]
            scale = np.sqrt(D) / (k_sel * k_sel).sum(-1, keepdim=True)           # [L, B, Hkv, 1]
            q = (k_sel * scale)[:, :, :, None, :] * peak[None, None, None, :, None]
            q = q.to(torch.bfloat16).reshape(L, B, Hq, D)
            slot_h = slot.cpu().numpy()
            # sampled units: the needle query rebuilt from the generator's key, not from the ring
            q_units = {}
            for u in units:
                l, b, h = u
                Ku, _ = unit_cache[u]
                kk = torch.as_tensor(Ku[slot_h[l, b, h]], dtype=torch.float32)
                qu = ((kk * (np.sqrt(D) / float((kk * kk).sum())))[None, :] * peak.cpu()[:, None]).to(torch.bfloat16)
                q[l, b, h * g:(h + 1) * g] = qu.to(dev)
                q_units[u] = np64(qu)
            out.zero_(); lse.zero_()
            cache.decode_attn(-1, q, out, None, lse)
            # every unit: output = the needle's value row, lse = the needle's logit (rings read back: a property)
            v_sel = Vr[li, bi, hi, slot].float()
            want = v_sel[:, :, :, None, :].expand(L, B, Hkv, g, D).reshape(L, B, Hq, D)
            qf = q.float().view(L, B, Hkv, g, D)
            logit = (qf * k_sel[:, :, :, None, :]).double().sum(-1) / np.sqrt(D)
            worst_all_out = max(worst_all_out, float((out.float() - want).abs().max()))
            worst_all_lse = max(worst_all_lse, float((lse.view(L, B, Hkv, g).double() - logit).abs().max()))
            assert worst_all_out <= TOL_OUT["bf16"], (T, i, worst_all_out)
            assert worst_all_lse <= 1e-3, (T, i, worst_all_lse)         # the other tokens add less than 1e-4
            # sampled units: float64 oracle on regenerated inputs
            out_h = np64(torch.stack([out[l, b, h * g:(h + 1) * g] for l, b, h in units]))
            lse_h = np64(torch.stack([lse[l, b, h * g:(h + 1) * g] for l, b, h in units]))
            for ui, u in enumerate(units):
                Ku, Vu = unit_cache[u]
                o_ref, lse_ref = attention_gqa(q_units[u], Ku[:, None, :], Vu[:, None, :])
                worst_out = max(worst_out, np.abs(out_h[ui] - o_ref).max())
                worst_lse = max(worst_lse, np.abs(lse_h[ui] - lse_ref).max())
                n_oracle += 1
    assert worst_out <= TOL_OUT["bf16"], worst_out
    assert worst_lse <= TOL_LSE["bf16"], worst_lse
    assert cache.status() == 0
    cache.close()
    torch.cuda.empty_cache()
    return info, n_oracle


@pytest.mark.parametrize("warps", [4, 3])
@pytest.mark.parametrize("W,B", [(333, 5), (1500, 7), (96, 3)])
def test_needle_in_every_tile_small_shapes(warps, W, B):
    """Both instantiations of the attention kernel; windows with a ragged last tile; rings that are partly filled,
    exactly full, and wrapped at an odd slot; most units split between CTAs (few units, 148 CTAs)."""
    c = {**CONFIGS["qwen7b"], "window": W, "batch": B}
    info, n = _run_needles(c, 2, [W - W // 3, W, W + W // 2 + 13], warps)
    assert info["consumer_warps"] == warps and n >= 5 * sum((min(T, W) + 31) // 32 for T in (W - W // 3, W, W + 1))


@pytest.mark.parametrize("name,warps", [("qwen7b", 0), ("qwen7b", 3), ("llama8b", 0)])
def test_needle_in_every_tile_full_size(name, warps):
    """The launch the benchmark times (all layers, full batch, full window): a needle in every unit at every tile
    position, for a ring that is not yet full and for one wrapped at an odd slot; the 7B shape on both
    instantiations of the kernel."""
    c = dict(CONFIGS[name])
    W = c["window"]
    info, n = _run_needles(c, c["n_layers"], [W - 301, W + 1013], warps)
    assert info["consumer_warps"] == (warps or 4)
    assert n >= 2 * (W // 32 - 10) * 5
