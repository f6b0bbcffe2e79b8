"""ptenc_attn_rings_static: attention over rings the caller owns, scratch inside the library image.

For users who cannot allocate device memory when they need attention (memory committed up front and the allocator
frozen, or a loop that must not hit the synchronisation an allocation implies): they cannot build a ptenc workspace,
so they hand their rings to this entry point.  The test builds such rings by hand, runs the entry point twice in a
row (the second call finds the first call's leftovers in the shared scratch) and compares each result with
ptenc_decode_attn on a regular cache holding the same tokens.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2602_16839_b200 as pt
from ptenc_inputs import SynthInputs

pytestmark = pytest.mark.gpu

TOL = 2e-2       # the bf16 output tolerance used throughout the GPU tests


def _rings_by_hand(gen, L, B, Hkv, D, W, T):
    """K/V rings as a caller would hold them: token t of every sequence sits in slot t mod W."""
    K = torch.zeros(L, B, Hkv, W, D, dtype=torch.bfloat16, device="cuda")
    V = torch.zeros_like(K)
    for t in range(T):
        k, v = gen.step_kv(t)
        K[:, :, :, t % W, :] = k
        V[:, :, :, t % W, :] = v
    count = min(T, W)
    head = (T - count) % W
    return K, V, head, count


@pytest.mark.parametrize("W,T", [(300, 170), (96, 250)])
def test_static_scratch_attention_matches_cache_path_twice(W, T):
    L, B, Hq, Hkv, D = 3, 6, 14, 2, 128
    shp = dict(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    gen = SynthInputs(seed=7, dtype="bf16", device="cuda", **shp)
    cfg = pt.make_config(window=W, dtype="bf16", **shp)
    cache = pt.Cache(cfg)
    for t in range(T):
        k, v = gen.step_kv(t)
        cache.append_evict(-1, k, v)
    K, V, head, count = _rings_by_hand(gen, L, B, Hkv, D, W, T)
    head_t = torch.full((L, B), head, dtype=torch.int32, device="cuda")
    count_t = torch.full((L, B), count, dtype=torch.int32, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for call in range(2):                                   # two calls in a row share the library's scratch
        q = gen.step_q(1000 + call)
        want = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device="cuda")
        lse_want = torch.zeros(L, B, Hq, dtype=torch.float32, device="cuda")
        cache.decode_attn(-1, q, want, None, lse_want)
        got = torch.zeros_like(want)
        lse_got = torch.zeros_like(lse_want)
        pt.attn_rings_static(cfg, K, V, head_t, count_t, q, got, None, lse_got, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert float((got.float() - want.float()).abs().max()) <= TOL
        assert float((lse_got - lse_want).abs().max()) <= 1e-4
        assert float(want.float().abs().max()) > 0.0
    assert cache.status() == 0
    cache.close()


def test_static_scratch_respects_active_mask_and_ragged_counts():
    L, B, Hq, Hkv, D, W = 2, 5, 8, 2, 64, 130
    shp = dict(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    gen = SynthInputs(seed=9, dtype="bf16", device="cuda", **shp)
    cfg = pt.make_config(window=W, dtype="bf16", **shp)
    K, V, _, _ = _rings_by_hand(gen, L, B, Hkv, D, W, W)
    counts = torch.tensor([[1, 40, 64, 65, 130], [130, 7, 0, 99, 33]], dtype=torch.int32, device="cuda")
    heads = torch.zeros_like(counts)
    active = torch.tensor([1, 1, 1, 0, 1], dtype=torch.uint8, device="cuda")
    q = gen.step_q(5)
    got = torch.full((L, B, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
    pt.attn_rings_static(cfg, K, V, heads, counts, q, got, active)
    torch.cuda.synchronize()
    g = Hq // Hkv
    for l in range(L):
        for b in range(B):
            n = int(counts[l, b])
            if not active[b] or n == 0:
                assert bool((got[l, b] == 7.0).all())            # untouched
                continue
            for h in range(Hq):
                kk = K[l, b, h // g, :n].float()
                vv = V[l, b, h // g, :n].float()
                p = torch.softmax(kk @ q[l, b, h].float() / D ** 0.5, dim=0)
                assert float((got[l, b, h].float() - p @ vv).abs().max()) <= TOL


def test_static_scratch_limits_are_errors():
    big = pt.make_config(n_layers=64, batch=512, n_q_heads=8, n_kv_heads=4, head_dim=128, window=8, dtype="bf16")
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    i = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(pt.PtencError) as e:
        pt.attn_rings_static(big, x, x, i, i, x, x)            # 131072 units > 65536: refused before any launch
    assert e.value.code == pt.binding.PTENC_ELIMIT
    fp32 = pt.make_config(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=1, head_dim=64, window=8, dtype="fp32")
    with pytest.raises(pt.PtencError) as e:
        pt.attn_rings_static(fp32, x, x, i, i, x, x)
    assert e.value.code == pt.binding.PTENC_ESHAPE
    torch.cuda.synchronize()
