"""ptenc_attn_rings_static: attention over rings the caller owns, scratch inside the library image.

For users who cannot allocate device memory when they need attention (memory committed up front and the allocator
frozen, or a loop that must not hit the synchronisation an allocation implies): they cannot build a ptenc workspace,
so they hand their rings to this entry point.  The tests build such rings by hand, run the entry point twice in a
row (the second call finds the first call's leftovers in the shared scratch) and compare each result with
ptenc_decode_attn on a regular cache holding the same tokens and with the float64 oracle on the same tokens; they
also watch the device's free memory and torch's allocator across the calls: nothing may be allocated.  Collected
last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2602_16839_b200 as pt
from oracle.ptenc_oracle import attention_gqa
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


@pytest.mark.parametrize("warps", [0, 3])
@pytest.mark.parametrize("W,T", [(300, 170), (96, 250)])
def test_static_scratch_attention_matches_cache_path_and_oracle_twice(W, T, warps):
    L, B, Hq, Hkv, D = 3, 6, 14, 2, 128
    shp = dict(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    gen = SynthInputs(seed=7, dtype="bf16", device="cuda", **shp)
    cfg = pt.make_config(window=W, dtype="bf16", attn_consumer_warps=warps, **shp)
    cache = pt.Cache(cfg)
    for t in range(T):
        k, v = gen.step_kv(t)
        cache.append_evict(-1, k, v)
    K, V, head, count = _rings_by_hand(gen, L, B, Hkv, D, W, T)
    head_t = torch.full((L, B), head, dtype=torch.int32, device="cuda")
    count_t = torch.full((L, B), count, dtype=torch.int32, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    live = list(range(T - count, T))                        # the tokens a window of W holds after T arrivals
    qs = [gen.step_q(1000 + call) for call in range(2)]
    want = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device="cuda")
    lse_want = torch.zeros(L, B, Hq, dtype=torch.float32, device="cuda")
    got = [torch.zeros_like(want) for _ in range(2)]
    lse_got = [torch.zeros_like(lse_want) for _ in range(2)]
    pt.attn_rings_static(cfg, K, V, head_t, count_t, qs[0], got[0], None, lse_got[0], status)   # per-device set-up
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for call in range(2):                                   # two calls in a row share the library's scratch
        got[call].zero_(); lse_got[call].zero_()
        pt.attn_rings_static(cfg, K, V, head_t, count_t, qs[call], got[call], None, lse_got[call], status)
    torch.cuda.synchronize()
    # nothing was allocated: not through torch's allocator, not behind its back
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert torch.cuda.mem_get_info()[0] >= free0
    assert int(status.item()) == 0
    for call in range(2):
        cache.decode_attn(-1, qs[call], want, None, lse_want)
        assert float((got[call].float() - want.float()).abs().max()) <= TOL
        assert float((lse_got[call] - lse_want).abs().max()) <= 1e-4
        assert float(want.float().abs().max()) > 0.0
        for l, b in ((0, 0), (L - 1, B - 1), (1, 2)):       # the oracle on the same tokens, regenerated
            Kl, Vl = gen.token_kv(l, b, live)
            o_ref, lse_ref = attention_gqa(qs[call][l, b].double().cpu().numpy(), Kl.double().numpy(),
                                           Vl.double().numpy())
            assert np.abs(got[call][l, b].double().cpu().numpy() - o_ref).max() <= TOL
            assert np.abs(lse_got[call][l, b].double().cpu().numpy() - lse_ref).max() <= 1e-4
    assert cache.status() == 0
    cache.close()


def test_static_scratch_reports_a_ring_state_out_of_range():
    """head/count come from the caller here: a count above the window (or a head outside it) is a bad value, not a
    fault -- that ring is skipped, its output rows stay as they were, and the status word says so (bit 2)."""
    L, B, Hq, Hkv, D, W = 1, 4, 8, 2, 128, 64
    shp = dict(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    gen = SynthInputs(seed=3, dtype="bf16", device="cuda", **shp)
    cfg = pt.make_config(window=W, dtype="bf16", **shp)
    K, V, _, _ = _rings_by_hand(gen, L, B, Hkv, D, W, W)
    counts = torch.tensor([[W, W + 1, 10, W]], dtype=torch.int32, device="cuda")
    heads = torch.tensor([[0, 0, 0, W]], dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q = gen.step_q(1)
    got = torch.full((L, B, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
    pt.attn_rings_static(cfg, K, V, heads, counts, q, got, None, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 2
    assert bool((got[0, 1] == 7.0).all()) and bool((got[0, 3] == 7.0).all())       # skipped
    for b, n in ((0, W), (2, 10)):                                                  # the good rings are served
        o_ref, _ = attention_gqa(q[0, b].double().cpu().numpy(), K[0, b, :, :n].transpose(0, 1).double().cpu().numpy(),
                                 V[0, b, :, :n].transpose(0, 1).double().cpu().numpy())
        assert np.abs(got[0, b].double().cpu().numpy() - o_ref).max() <= TOL
    # the next call starts from a clean status word
    counts[0, 1], heads[0, 3] = W, 0
    pt.attn_rings_static(cfg, K, V, heads, counts, q, got, None, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and not bool((got == 7.0).any())


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
