"""GPU parity: the CUDA path through the C ABI vs the CPU oracle, same seeded inputs."""
import numpy as np
import pytest
import torch

import paper_2602_16839_b200 as pt
from ptenc_inputs import CONFIGS

from _harness import TOL_LSE, TOL_OUT, TOL_STATE, Pair, np64

pytestmark = pytest.mark.gpu


def _cfg(name):
    c = dict(CONFIGS[name])
    steps = c.pop("steps")
    c.pop("ragged", None)
    return c, steps


def test_tiny_fp32_exhaustive():
    """Configuration 1 whole: every step, sequence and head; ring state bit-exact; state within tolerance."""
    c, steps = _cfg("tiny")
    p = Pair(pt, seed=0, **c)
    B = c["batch"]
    slot = torch.empty(B, dtype=torch.int32, device="cuda")
    first = torch.empty(B, dtype=torch.int64, device="cuda")
    nev = torch.empty(B, dtype=torch.int32, device="cuda")
    lse = torch.empty(B, c["n_q_heads"], dtype=torch.float32, device="cuda")
    out = torch.empty(B, c["n_q_heads"], c["head_dim"], dtype=torch.float32, device="cuda")
    worst = 0.0
    for t in range(steps):
        q = p.gen.step_q(t)
        k, v = p.gen.step_kv(t)
        p.cache.append_evict(0, k[0], v[0], None, slot, first, nev)
        p.cache.encode(0)
        p.cache.decode_attn(0, q[0], out, None, lse)
        o_ref, lse_ref, (slots, ev_t, ev_s) = p.orc.decode_step(0, np64(q[0]), np64(k[0]), np64(v[0]))
        assert np.array_equal(slot.cpu().numpy(), slots)
        want_first = [e[0] if e else -1 for e in ev_t]
        assert first.cpu().tolist() == want_first and nev.cpu().tolist() == [len(e) for e in ev_t]
        worst = max(worst, np.abs(np64(out) - o_ref).max())
        assert np.abs(np64(lse) - lse_ref).max() <= TOL_LSE["fp32"]
        p.check_ring()
        if t % 16 == 0 or t == steps - 1:
            p.check_state()
    assert worst <= TOL_OUT["fp32"], worst
    assert p.cache.status() == 0
    p.close()


# storage dtype and, for bf16, the consumer-warp count of the tensor-core attention kernel: 0 = the default (four),
# 3 = the other instantiation
KERNELS = [("fp32", 0), ("bf16", 0), ("bf16", 3)]


@pytest.mark.parametrize("dtype,warps", KERNELS)
@pytest.mark.parametrize("Hq,Hkv", [(1, 1), (4, 1), (7, 1), (8, 2), (14, 2), (12, 3)])
def test_small_shapes_ragged(dtype, warps, Hq, Hkv):
    """Query-group sizes 1,4,7,8; window not a power of two; sequences active at random."""
    rng = np.random.default_rng(Hq * 10 + Hkv)
    p = Pair(pt, n_layers=2, batch=5, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=64 if dtype == "fp32" else 128,
             window=37, evict_chunk=1, dtype=dtype, seed=3, attn_consumer_warps=warps)
    for t in range(37 * 2 + 11):
        active = (rng.random(5) < 0.8).astype(np.uint8)
        if t == 0:
            active[:] = [1, 1, 0, 1, 0]
        p.step(t, active=active)
        if t % 9 == 0:
            p.check_ring()
    p.check_ring()
    p.check_state()
    assert p.cache.status() == 0
    p.close()


@pytest.mark.parametrize("dtype,warps", KERNELS)
@pytest.mark.parametrize("W,E", [(1, 1), (2, 1), (3, 2), (5, 5), (64, 16), (100, 25), (100, 100), (130, 1), (257, 65)])
def test_windows_and_chunks(dtype, warps, W, E):
    """E in {1, ceil(W/4), W}; W = 1 returns v of the newest token; ragged tile tails."""
    p = Pair(pt, n_layers=1, batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128 if dtype == "bf16" else 32,
             window=W, evict_chunk=E, dtype=dtype, seed=W, attn_consumer_warps=warps)
    T = min(3 * W + 5, 2 * W + 70)
    for t in range(T):
        p.step(t)
        if W == 1:
            _, v = p.gen.step_kv(t)
            want = v[0].repeat_interleave(4, dim=1)
            assert torch.equal(p.out[0], want)
    p.check_ring()
    p.check_state()
    assert p.cache.status() == 0
    p.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("E,batch", [(3, 4), (1, 4), (1, 21)])
def test_fused_step_equals_three_calls(dtype, E, batch):
    kw = dict(n_layers=3, batch=batch, n_q_heads=8, n_kv_heads=2, head_dim=128, window=70, evict_chunk=E,
              dtype=dtype, seed=5)
    a, b, c = Pair(pt, **kw), Pair(pt, **kw), Pair(pt, **kw)
    for t in range(160):
        a.step(t, fused=True, all_layers=True)
        b.step(t, fused=False, all_layers=True)
        c.step(t, fused=True, all_layers=False)
        assert torch.equal(a.out, b.out)
        # per-layer calls split the tiles between CTAs at other points than the all-layer call does, so the fp32
        # partial sums are combined in another order: equal to within a few bf16 ulps, not bit for bit
        assert float((a.out.float() - c.out.float()).abs().max()) <= 4e-3
    for l in range(3):
        assert torch.equal(a.cache.get_state(l), b.cache.get_state(l))
        assert torch.equal(a.cache.get_state(l), c.cache.get_state(l))
    a.check_state(); a.check_ring()
    for x in (a, b, c):
        x.close()


@pytest.mark.parametrize("warps", [0, 3])
def test_bf16_multi_tile_lse(warps):
    """Several 32-token tiles plus a tail, all query heads of a 7-group, lse output."""
    p = Pair(pt, n_layers=2, batch=3, n_q_heads=28, n_kv_heads=4, head_dim=128, window=333, dtype="bf16", seed=11,
             n_global=32, rank=32, attn_consumer_warps=warps)
    lse = torch.empty(2, 3, 28, dtype=torch.float32, device="cuda")
    for t in range(333 + 80):
        p.step(t)
        if t in (0, 63, 64, 200, 332, 333, 400):
            q = p.gen.step_q(t)
            p.cache.decode_attn(-1, q, p.out, None, lse)
            for l in range(2):
                o_ref, lse_ref = p.orc.decode_attn(l, np64(q[l]))
                assert np.abs(np64(p.out[l]) - o_ref).max() <= TOL_OUT["bf16"]
                assert np.abs(np64(lse[l]) - lse_ref).max() <= TOL_LSE["bf16"]
    p.check_state(); p.check_ring()
    assert p.cache.status() == 0
    p.close()


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_normalize_modes_and_ablations(mode):
    kw = dict(n_layers=1, batch=3, n_q_heads=4, n_kv_heads=2, head_dim=64, window=9, dtype="bf16", seed=mode)
    # mode 2 never normalises: compare relative to the state's magnitude
    p = Pair(pt, normalize_mode=mode, **kw)
    for t in range(60):
        p.step(t)
    p.check_state(rel=(mode == 2))
    p.close()
    # Global-Only: the state never leaves S_0 (Sec. 4.3 ablation)
    p = Pair(pt, normalize_mode=mode, encode_enabled=0, **kw)
    s0 = p.cache.get_state(0).clone()
    for t in range(30):
        p.step(t)
    assert torch.equal(p.cache.get_state(0), s0)
    p.check_state()
    p.close()
    # #Global-0: zero start
    p = Pair(pt, normalize_mode=mode, global_kv=False, **kw)
    assert float(p.cache.get_state(0).abs().max()) == 0.0
    for t in range(30):
        p.step(t)
    p.check_state(rel=(mode == 2))
    p.close()


def test_encode_with_caller_rows():
    """ptenc_encode on rows supplied by the caller, ragged n_evicted, and state size independent of m."""
    p = Pair(pt, n_layers=2, batch=4, n_q_heads=8, n_kv_heads=2, head_dim=64, window=8, dtype="bf16", seed=2,
             n_global=16, rank=24)
    m_max, d_kv = 11, 128
    Ke = p.gen.generic(40, 0, (2, 4, m_max, d_kv), 1.0)
    Ve = p.gen.generic(41, 0, (2, 4, m_max, d_kv), 1.0)
    n_ev = torch.tensor([[0, 1, 11, 5], [3, 0, 0, 7]], dtype=torch.int32, device="cuda")
    p.cache.encode(-1, Ke, Ve, n_ev, m_max)
    for l in range(2):
        rowsK = [np64(Ke[l, b, :n_ev[l, b]]) for b in range(4)]
        rowsV = [np64(Ve[l, b, :n_ev[l, b]]) for b in range(4)]
        p.orc.encode(l, rowsK, rowsV)
        assert p.cache.get_state(l).shape == (4, 16, 24)
    p.check_state()
    # single layer call
    p.cache.encode(1, Ke[1], Ve[1], n_ev[1], m_max)
    p.orc.encode(1, [np64(Ke[1, b, :n_ev[1, b]]) for b in range(4)], [np64(Ve[1, b, :n_ev[1, b]]) for b in range(4)])
    p.check_state()
    p.close()


def test_reset_with_mask():
    p = Pair(pt, n_layers=2, batch=3, n_q_heads=4, n_kv_heads=1, head_dim=64, window=6, dtype="fp32", seed=8)
    for t in range(15):
        p.step(t)
    mask = torch.tensor([1, 0, 1], dtype=torch.uint8, device="cuda")
    s_before = p.cache.get_state(0).clone()
    p.cache.reset(mask)
    head, count, n_app = p.cache.get_ring(1)
    assert count.tolist() == [0, 6, 0] and n_app.tolist() == [0, 15, 0]
    s_after = p.cache.get_state(0)
    assert torch.equal(s_after[1], s_before[1])
    P = p.gen.encoder_params(0)
    from oracle.ptenc_oracle import initial_state, latent_queries
    Qa = latent_queries(np64(P["Wq_a"]), np64(P["q_g"]))
    S0 = initial_state(Qa, np64(P["Wk_a"]), np64(P["Wv_a"]), np64(P["k_g"]), np64(P["v_g"]))
    assert np.abs(np64(s_after[0]) - S0).max() <= 1e-4 * max(1.0, np.abs(S0).max())
    p.close()


def test_error_paths_on_device_box():
    cfg = pt.make_config(n_layers=1, batch=2, n_q_heads=4, n_kv_heads=1, head_dim=64, window=8, dtype="bf16")
    c = pt.Cache(cfg)
    x = torch.zeros(2, 4, 64, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(2, 1, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pt.PtencError) as e:
        c.decode_step(1, x, kv, kv, x)
    assert e.value.code == pt.binding.PTENC_EINVAL
    with pytest.raises(pt.PtencError) as e:
        c.decode_step(0, x.view(-1)[1:], kv, kv, x)       # 2-byte offset: misaligned
    assert e.value.code == pt.binding.PTENC_EALIGN
    with pytest.raises(pt.PtencError):
        c.decode_attn(0, None, x)
    assert c.status() == 0
    c.close()


def test_tensor_core_kernel_serves_bf16_shapes():
    """The TMA + tensor-core kernel (not the generic one) is the path taken for the paper-shaped configs."""
    for name in ("qwen3b", "qwen7b", "llama8b"):
        c = dict(CONFIGS[name])
        cfg = pt.make_config(n_layers=1, batch=2, n_q_heads=c["n_q_heads"], n_kv_heads=c["n_kv_heads"],
                             head_dim=c["head_dim"], window=128, dtype="bf16")
        cache = pt.Cache(cfg)
        info = cache.info()
        assert info["tensor_core_attn"] and info["attn_grid"] >= 100
        cache.close()
    cache = pt.Cache(pt.make_config(n_layers=1, batch=2, n_q_heads=4, n_kv_heads=1, head_dim=64, window=64,
                                    dtype="fp32"))
    assert not cache.info()["tensor_core_attn"]
    cache.close()


@pytest.mark.parametrize("warps", [0, 3])
def test_split_units_many_tiles_per_cta(warps):
    """Enough tiles that every CTA streams many pipeline rounds and most units are split between CTAs."""
    p = Pair(pt, n_layers=2, batch=7, n_q_heads=28, n_kv_heads=4, head_dim=128, window=1500, dtype="bf16", seed=21,
             attn_consumer_warps=warps)
    # fill quickly: same synthetic stream on both sides, outputs checked at chosen steps only
    for t in range(1500 + 30):
        chk = t in (0, 1, 63, 64, 65, 700, 1499, 1500, 1501, 1529)
        if chk:
            p.step(t)
        else:
            q = p.gen.step_q(t)
            k, v = p.gen.step_kv(t)
            p.cache.decode_step(-1, q, k, v, p.out)
            for l in range(2):
                p.orc.append_evict(l, np64(k[l]), np64(v[l]))
                p.orc.encode(l)
    p.check_ring(); p.check_state()
    assert p.cache.status() == 0
    p.close()


@pytest.mark.parametrize("W,E,G,r,Hkv", [(64, 16, 32, 32, 2), (600, 150, 32, 32, 4), (256, 128, 16, 16, 2),
                                         (300, 129, 48, 64, 2), (40, 5, 8, 32, 1), (2048, 512, 32, 32, 4)])
def test_chunk_eviction_on_the_tensor_core_encoder(W, E, G, r, Hkv):
    """Chunks of E tokens leave at once (Sec. 4.1: 25 % of the window in the paper's runs): the projections run on
    tcgen05; tiles of 128 tokens with ragged tails, every supported rank, state against the float64 oracle."""
    p = Pair(pt, n_layers=2, batch=3, n_q_heads=2 * Hkv, n_kv_heads=Hkv, head_dim=128, window=W, evict_chunk=E,
             dtype="bf16", seed=W + E, n_global=G, rank=r)
    assert p.cache.info()["tensor_core_encode"]
    T = W + 2 * E + 3
    checks = {0, W - 1, W, W + 1, W + E - 1, W + E, W + E + 1, T - 1}
    states_at = {W, W + E, T - 1}
    for t in range(T):
        if t in checks:
            p.step(t)
        else:
            q = p.gen.step_q(t)
            k, v = p.gen.step_kv(t)
            p.cache.decode_step(-1, q, k, v, p.out)
            for l in range(p.L):
                p.orc.append_evict(l, np64(k[l]), np64(v[l]))
                p.orc.encode(l)
        if t in states_at:
            p.check_state()
            p.check_ring()
    assert p.cache.status() == 0
    p.close()


def test_tensor_core_encoder_with_caller_rows_and_modes():
    """ptenc_encode on caller-supplied chunks: ragged row counts around the 128-row tile, all three Normalize modes."""
    for mode in (0, 1, 2):
        p = Pair(pt, n_layers=2, batch=6, n_q_heads=8, n_kv_heads=4, head_dim=64, window=16, evict_chunk=4,
                 dtype="bf16", seed=40 + mode, n_global=24, rank=32, normalize_mode=mode)
        assert p.cache.info()["tensor_core_encode"]
        m_max, d_kv = 200, 256
        Ke = p.gen.generic(40, 0, (2, 6, m_max, d_kv), 1.0)
        Ve = p.gen.generic(41, 0, (2, 6, m_max, d_kv), 1.0)
        n_ev = torch.tensor([[0, 1, 127, 128, 129, 200], [200, 64, 0, 7, 130, 255]], dtype=torch.int32, device="cuda")
        for rep in range(2):
            p.cache.encode(-1, Ke, Ve, n_ev, m_max)
            for l in range(2):
                cnt = [min(int(n_ev[l, b]), m_max) for b in range(6)]
                p.orc.encode(l, [np64(Ke[l, b, :cnt[b]]) for b in range(6)], [np64(Ve[l, b, :cnt[b]]) for b in range(6)])
            p.check_state(rel=(mode == 2), tol=2e-4 if mode == 2 else TOL_STATE)
        assert p.cache.status() == 0
        p.close()


@pytest.mark.parametrize("dtype,L", [("bf16", 9), ("fp32", 2)])
def test_host_buffer_step_equals_device_step(dtype, L):
    """ptenc_decode_step_host (pinned host tensors in and out, copies overlapped on internal streams) gives the same
    outputs, ring and state as ptenc_decode_step on device tensors; also with a mask and for a single layer."""
    kw = dict(n_layers=L, batch=5, n_q_heads=8, n_kv_heads=2, head_dim=128 if dtype == "bf16" else 64, window=23,
              evict_chunk=1, dtype=dtype, seed=31)
    a, b = Pair(pt, **kw), Pair(pt, **kw)
    staging = torch.empty(b.cache.host_staging_bytes(-1), dtype=torch.uint8, device="cuda")
    hout = torch.zeros(a.out.shape, dtype=a.out.dtype).pin_memory()
    rng = np.random.default_rng(3)
    for t in range(60):
        active = (rng.random(5) < 0.85).astype(np.uint8) if t % 3 else None
        a.step(t, active=active)
        q = b.gen.step_q(t)
        k, v = b.gen.step_kv(t)
        qh, kh, vh = (x.cpu().pin_memory() for x in (q, k, v))
        ah = None if active is None else torch.as_tensor(active).pin_memory()
        if t % 7 == 5:                                   # layer by layer through the same entry point
            for l in range(L):
                b.cache.decode_step_host(l, qh[l], kh[l], vh[l], hout[l], staging, ah)
        else:
            b.cache.decode_step_host(-1, qh, kh, vh, hout, staging, ah)
        torch.cuda.synchronize()
        m = np.ones(5, bool) if active is None else active.astype(bool)
        got, want = hout[:, m].float(), a.out[:, m].cpu().float()
        assert float((got - want).abs().max()) <= (4e-3 if dtype == "bf16" else 1e-6)
    for l in range(L):
        assert torch.equal(a.cache.get_state(l), b.cache.get_state(l))
        for x, y in zip(a.cache.get_ring(l), b.cache.get_ring(l)):
            assert torch.equal(x, y)
    assert a.cache.status() == 0 and b.cache.status() == 0
    a.close(); b.close()


@pytest.mark.parametrize("dtype,warps", KERNELS)
@pytest.mark.parametrize("W,E,prompts", [(37, 1, [0, 1, 17, 36, 5]), (96, 24, [0, 33, 64, 95, 80]),
                                         (200, 50, [130, 7, 0, 199, 64])])
def test_pinned_prompt_and_sliding_window_over_the_rest(dtype, warps, W, E, prompts):
    """Prompt lengths from none to W - 1 (a single sliding slot), chunks larger than the remaining capacity, tiles
    that straddle the end of the pinned part: outputs, eviction reports, ring and state against the oracle."""
    p = Pair(pt, n_layers=2, batch=5, n_q_heads=8, n_kv_heads=2, head_dim=128 if dtype == "bf16" else 64,
             window=W, evict_chunk=E, dtype=dtype, seed=W, n_global=16, rank=16, attn_consumer_warps=warps)
    p.prefill(prompts, max(prompts))
    p.check_ring()
    B = 5
    slot = torch.empty(B, dtype=torch.int32, device="cuda")
    first = torch.empty(B, dtype=torch.int64, device="cuda")
    nev = torch.empty(B, dtype=torch.int32, device="cuda")
    out1 = torch.zeros(B, 8, p.D, dtype=p.cache.torch_dtype, device="cuda")
    for t in range(2 * W + 9):
        if t % 4 == 3:                                    # three separate calls on layer 1, index reports checked
            q = p.gen.step_q(t)
            k, v = p.gen.step_kv(t)
            p.cache.decode_step(0, q[0], k[0], v[0], p.out[0])
            p.cache.append_evict(1, k[1], v[1], None, slot, first, nev)
            p.cache.encode(1)
            p.cache.decode_attn(1, q[1], out1)
            for l in range(2):
                o_ref, _, (slots, ev_t, ev_s) = p.orc.decode_step(l, np64(q[l]), np64(k[l]), np64(v[l]))
                got = p.out[0] if l == 0 else out1
                assert np.abs(np64(got) - o_ref).max() <= TOL_OUT[dtype]
            assert np.array_equal(slot.cpu().numpy(), slots)
            assert first.cpu().tolist() == [e[0] if e else -1 for e in ev_t]
            assert nev.cpu().tolist() == [len(e) for e in ev_t]
        else:
            p.step(t)
        if t % 11 == 0:
            p.check_ring()
    p.check_ring()
    p.check_state()
    assert p.cache.status() == 0
    p.close()


def test_prefill_misuse_sets_the_status_word():
    p = Pair(pt, n_layers=1, batch=3, n_q_heads=4, n_kv_heads=1, head_dim=64, window=8, dtype="bf16", seed=1)
    p.step(0)                                              # sequences are no longer empty
    Kp = torch.zeros(1, 3, 8, 1, 64, dtype=torch.bfloat16, device="cuda")
    n = torch.tensor([2, 0, 0], dtype=torch.int32, device="cuda")
    p.cache.prefill(-1, Kp, Kp, n, 8)
    assert p.cache.status() == 2 and p.cache.get_pinned(0).tolist() == [0, 0, 0]
    p.cache.reset()                                        # clears rings, pinned counts and the status word
    assert p.cache.status() == 0
    n = torch.tensor([8, 3, 0], dtype=torch.int32, device="cuda")      # 8 = W: no slot left for the sliding part
    p.cache.prefill(-1, Kp, Kp, n, 8)
    assert p.cache.status() == 2 and p.cache.get_pinned(0).tolist() == [0, 3, 0]
    p.close()


@pytest.mark.parametrize("dtype,G,r,d_in,d_out,B", [("bf16", 16, 24, 328, 200, 11), ("fp32", 16, 24, 328, 200, 11),
                                                    ("bf16", 32, 32, 352, 200, 11), ("bf16", 64, 16, 1024, 520, 11),
                                                    ("bf16", 32, 32, 1792, 904, 37), ("bf16", 64, 64, 512, 264, 20),
                                                    ("bf16", 128, 16, 256, 72, 16), ("bf16", 96, 32, 3584, 64, 130)])
def test_dynamic_weight_update_from_the_running_state(dtype, G, r, d_in, d_out, B):
    """y += A (S (B x)) with the state the rollout has produced so far, per sequence, against the oracle's
    (W + A S B) x written out; masked rows untouched; all layers in one call and one layer alone."""
    from oracle.ptenc_oracle import lora_apply
    L = 2             # the first two shape sets take the shape-generic kernel, the others the tensor-core kernels
    p = Pair(pt, n_layers=L, batch=B, n_q_heads=4, n_kv_heads=2, head_dim=64, window=12, evict_chunk=3, dtype=dtype,
             seed=77, n_global=G, rank=r)
    for t in range(30):
        p.step(t)
    A = p.gen.generic(60, 0, (L, d_out, G), G ** -0.5)
    Bm = p.gen.generic(61, 0, (L, r, d_in), d_in ** -0.5)
    x = p.gen.generic(62, 0, (L, B, d_in), 1.0)
    y0 = p.gen.generic(63, 0, (L, B, d_out), 1.0)
    active = torch.tensor([0 if b % 7 == 2 else 1 for b in range(B)], dtype=torch.uint8, device="cuda")
    y = y0.clone()
    p.cache.lora_apply(-1, A, Bm, x, y, active)
    y1 = y0[1].clone()
    p.cache.lora_apply(1, A[1], Bm[1], x[1], y1)
    m = active.bool().cpu().numpy()
    tol = 2e-2 if dtype == "bf16" else 2e-5
    for l in range(L):
        ref = lora_apply(np64(y0[l]), np64(x[l]), np64(A[l]), p.orc.S[l], np64(Bm[l]))
        got = np64(y[l])
        assert np.abs(got[m] - ref[m]).max() <= tol
        assert np.array_equal(got[~m], np64(y0[l])[~m])
        assert np.abs(ref - np64(y0[l])).max() > 0.05            # the update is not a no-op
    assert np.abs(np64(y1) - lora_apply(np64(y0[1]), np64(x[1]), np64(A[1]), p.orc.S[1], np64(Bm[1]))).max() <= tol
    assert p.cache.status() == 0
    p.close()


@pytest.mark.parametrize("warps", [0, 3])
@pytest.mark.parametrize("W,E,prompts", [(150, 1, [0, 70, 149]), (300, 75, [64, 0, 130])])
def test_head_dim_64_tensor_core_attention_with_pinned_prompt(warps, W, E, prompts):
    """The D = 64 variant of the TMA attention kernel (64-token tiles), several tiles, pinned entries that end inside
    a tile, group size 7."""
    p = Pair(pt, n_layers=2, batch=3, n_q_heads=14, n_kv_heads=2, head_dim=64, window=W, evict_chunk=E, dtype="bf16",
             seed=W + 1, n_global=16, rank=16, attn_consumer_warps=warps)
    assert p.cache.info()["tensor_core_attn"]
    p.prefill(prompts, max(prompts))
    for t in range(W + 2 * E + 30):
        if t % 5 == 0 or t > W - 3:
            p.step(t)
        else:
            q = p.gen.step_q(t)
            k, v = p.gen.step_kv(t)
            p.cache.decode_step(-1, q, k, v, p.out)
            for l in range(p.L):
                p.orc.append_evict(l, np64(k[l]), np64(v[l]))
                p.orc.encode(l)
    p.check_ring(); p.check_state()
    assert p.cache.status() == 0
    p.close()


def test_host_buffer_steps_back_to_back_without_synchronising():
    """Six host-buffer steps enqueued with no synchronisation in between (the uploads of a step overlap the kernels of
    the step before, two staging halves in turn), each with its own host buffers: every output equals the device
    path's."""
    kw = dict(n_layers=6, batch=9, n_q_heads=8, n_kv_heads=2, head_dim=128, window=40, evict_chunk=1, dtype="bf16",
              seed=61)
    a, b = Pair(pt, **kw), Pair(pt, **kw)
    for t in range(45):                                     # rings full, evicting
        a.step(t); b.step(t, check=False)
    staging = torch.empty(b.cache.host_staging_bytes(-1), dtype=torch.uint8, device="cuda")
    steps = range(45, 51)
    host_in, host_out, want = [], [], []
    for t in steps:
        q = b.gen.step_q(t)
        k, v = b.gen.step_kv(t)
        host_in.append(tuple(x.cpu().pin_memory() for x in (q, k, v)))
        host_out.append(torch.zeros(a.out.shape, dtype=a.out.dtype).pin_memory())
    torch.cuda.synchronize()
    for i, t in enumerate(steps):
        b.cache.decode_step_host(-1, *host_in[i], host_out[i], staging)
    torch.cuda.synchronize()
    for i, t in enumerate(steps):
        a.step(t)
        assert float((host_out[i].float() - a.out.cpu().float()).abs().max()) <= 4e-3
    for l in range(6):
        assert torch.equal(a.cache.get_state(l), b.cache.get_state(l))
    assert b.cache.status() == 0
    a.close(); b.close()


@pytest.mark.parametrize("E", [1, 3])
@pytest.mark.parametrize("G,r", [(5, 12), (3, 40), (128, 128)])
def test_odd_state_shapes_take_the_right_encoder(G, r, E):
    """Ranks that are not a multiple of 8 (shape-generic encoder), a rank of 40 (warp-mma kernel for E = 1, generic for
    chunks), and the largest state (128 x 128: four values of a state row per lane)."""
    p = Pair(pt, n_layers=2, batch=3, n_q_heads=4, n_kv_heads=2, head_dim=64, window=11, evict_chunk=E, dtype="bf16",
             seed=G + r + E, n_global=G, rank=r)
    for t in range(40):
        p.step(t)
    p.check_state()
    p.check_ring()
    assert p.cache.status() == 0
    p.close()


@pytest.mark.parametrize("dtype,E", [("bf16", 1), ("bf16", 8), ("fp32", 1)])
def test_sequences_finish_and_their_places_are_reused(dtype, E):
    """A rollout batch in which sequences end at different times: a finished sequence is reset, a new prompt is
    pinned in its place, and it decodes on beside the others (which are in the middle of their windows)."""
    B, W = 6, 40
    p = Pair(pt, n_layers=2, batch=B, n_q_heads=8, n_kv_heads=2, head_dim=128 if dtype == "bf16" else 64, window=W,
             evict_chunk=E, dtype=dtype, seed=90 + E, n_global=16, rank=16)
    p.prefill([5, 0, 12, 30, 0, 39], 39)
    rng = np.random.default_rng(4)
    for t in range(150):
        if t in (37, 61, 90, 133):                          # some sequences finish; new ones take their places
            done = (rng.random(B) < 0.4).astype(np.uint8)
            done[t % B] = 1
            p.cache.reset(torch.as_tensor(done, device="cuda"))
            p.orc.reset(done)
            n_new = np.where(done, rng.integers(0, W, B), 0)
            p.prefill(n_new.tolist(), max(1, int(n_new.max())), tensor_id=70 + t)
            p.check_ring()
        p.step(t)
    p.check_ring()
    p.check_state()
    assert p.cache.status() == 0
    p.close()


def test_reset_clears_stale_split_unit_counters_and_status():
    """A launch that gives up part-way can leave arrival counts of split units behind.  Stand-in for that (no fault
    is provoked): non-zero counters and a status word are written into the workspace by hand; after the full reset
    attention over freshly filled rings is right again -- with stale counters the last-arriver test of a split unit
    would fire early or never."""
    p = Pair(pt, n_layers=2, batch=7, n_q_heads=28, n_kv_heads=4, head_dim=128, window=700, dtype="bf16", seed=33)
    ptr_t, n_t = p.cache.workspace_region(pt.binding.REGION_TICKETS)
    ptr_s, n_s = p.cache.workspace_region(pt.binding.REGION_STATUS)
    base = p.cache.workspace.data_ptr()
    tickets = p.cache.workspace[ptr_t - base: ptr_t - base + n_t].view(torch.int32)
    status = p.cache.workspace[ptr_s - base: ptr_s - base + n_s].view(torch.int32)
    assert tickets.numel() == 2 * 7 * 4 and int(tickets.abs().max()) == 0
    tickets.copy_(torch.arange(1, tickets.numel() + 1, dtype=torch.int32, device="cuda") % 3 + 1)
    status.fill_(1)
    assert p.cache.status() == 1
    p.cache.reset()
    p.orc.reset()
    assert p.cache.status() == 0 and int(tickets.abs().max()) == 0
    for t in range(700 + 5):
        if t in (0, 31, 32, 699, 700, 704):
            p.step(t)
        else:
            q = p.gen.step_q(t)
            k, v = p.gen.step_kv(t)
            p.cache.decode_step(-1, q, k, v, p.out)
            for l in range(2):
                p.orc.append_evict(l, np64(k[l]), np64(v[l]))
                p.orc.encode(l)
    assert int(tickets.abs().max()) == 0            # the counters clean themselves after every launch
    p.check_ring(); p.check_state()
    assert p.cache.status() == 0
    p.close()


def test_launch_info_reports_the_instantiation():
    """Four consumer warps unless the configuration asks for three."""
    c7 = dict(CONFIGS["qwen7b"])
    kw = dict(n_q_heads=c7["n_q_heads"], n_kv_heads=c7["n_kv_heads"], head_dim=128, dtype="bf16")
    small = pt.Cache(pt.make_config(n_layers=2, batch=2, window=2048, **kw))
    assert small.attn_launch_info(-1) == {"consumer_warps": 4, "tile_tokens": 32, "stages": 12}
    small.close()
    forced = pt.Cache(pt.make_config(n_layers=2, batch=2, window=2048, attn_consumer_warps=3, **kw))
    assert forced.attn_launch_info(-1)["consumer_warps"] == 3 and forced.attn_launch_info(0)["consumer_warps"] == 3
    forced.close()
    d64 = pt.Cache(pt.make_config(n_layers=1, batch=2, n_q_heads=8, n_kv_heads=2, head_dim=64, window=256, dtype="bf16"))
    assert d64.attn_launch_info(-1) == {"consumer_warps": 4, "tile_tokens": 64, "stages": 12}
    d64.close()
    gen = pt.Cache(pt.make_config(n_layers=1, batch=2, n_q_heads=4, n_kv_heads=1, head_dim=64, window=64, dtype="fp32"))
    assert gen.attn_launch_info(-1) == {"consumer_warps": 0, "tile_tokens": 0, "stages": 0}
    gen.close()


def test_a_step_with_every_sequence_inactive_changes_nothing_and_leaves_the_counters_clean():
    """A launch with no work at all (every sequence masked out): outputs untouched, rings and states unchanged, status
    clean -- and the launches after it behave as if it had not happened (the attention kernel's work counter and its
    split-unit tickets are back at zero), on both instantiations."""
    for warps in (0, 3):
        p = Pair(pt, n_layers=2, batch=5, n_q_heads=8, n_kv_heads=2, head_dim=128, window=40, dtype="bf16", seed=9,
                 attn_consumer_warps=warps)
        for t in range(44):
            p.step(t)
        S_before = [p.cache.get_state(l).clone() for l in range(2)]
        ring_before = [tuple(x.clone() for x in p.cache.get_ring(l)) for l in range(2)]
        q = p.gen.step_q(44)
        k, v = p.gen.step_kv(44)
        out = torch.full_like(q, 7.0)
        none = torch.zeros(5, dtype=torch.uint8, device="cuda")
        p.cache.decode_step(-1, q, k, v, out, none)
        assert torch.equal(out, torch.full_like(q, 7.0))
        for l in range(2):
            assert torch.equal(p.cache.get_state(l), S_before[l])
            assert all(torch.equal(a, b) for a, b in zip(p.cache.get_ring(l), ring_before[l]))
        assert p.cache.status() == 0
        for t in range(44, 50):                            # ordinary steps afterwards, checked against the oracle
            p.step(t)
        assert p.cache.status() == 0
        p.close()


@pytest.mark.parametrize("warps", [0, 3])
def test_item_lookup_by_arithmetic_and_by_search_give_the_same_bits(warps):
    """The attention kernel finds the (layer, sequence, head) of a work item by arithmetic when every sequence of the
    call has tokens and no unit is split, and by a search over prefix sums otherwise.  Masking one sequence out
    switches a launch from the first way to the second; the other sequences' outputs and log-sum-exps must not
    change by a bit (nor does it matter which CTA a work item lands on)."""
    L, B, Hq = 2, 6, 8
    p = Pair(pt, n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=2, head_dim=128, window=200, dtype="bf16", seed=21,
             attn_consumer_warps=warps)
    for t in range(230):
        p.step(t, check=(t % 50 == 0))
    q = p.gen.step_q(230)
    out_a = torch.zeros(L, B, Hq, 128, dtype=torch.bfloat16, device="cuda")
    out_b = torch.full_like(out_a, 3.0)
    lse_a = torch.zeros(L, B, Hq, dtype=torch.float32, device="cuda")
    lse_b = torch.full_like(lse_a, 3.0)
    p.cache.decode_attn(-1, q, out_a, None, lse_a)
    for masked in (0, 3, B - 1):
        act = torch.ones(B, dtype=torch.uint8, device="cuda")
        act[masked] = 0
        out_b.fill_(3.0)
        lse_b.fill_(3.0)
        p.cache.decode_attn(-1, q, out_b, act, lse_b)
        keep = [b for b in range(B) if b != masked]
        assert torch.equal(out_a[:, keep], out_b[:, keep])
        assert torch.equal(lse_a[:, keep], lse_b[:, keep])
        assert torch.equal(out_b[:, masked], torch.full_like(out_b[:, masked], 3.0))      # not written
    assert p.cache.status() == 0
    p.close()
