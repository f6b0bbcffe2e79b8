"""Pins for the CPU oracle: closed forms, invariants, library routines, brute force.

None of these re-types the oracle's own formula with the oracle's own primitives:
ring indices are checked against closed forms and a naive list model, attention
against torch's scaled-dot-product routine and special cases with known answers,
the encoder against exact rational arithmetic in pure Python, a hand-worked integer
example, and algebraic identities.
"""
import importlib
import itertools
import os
import types
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle.ptenc_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))


# =====================================================================================
# pins are functions of the oracle module so that a mutated copy can be run through them
# =====================================================================================
def _mk(mod, **kw):
    base = dict(n_layers=1, batch=1, n_q_heads=2, n_kv_heads=1, head_dim=4, window=4,
                evict_chunk=1, n_global=3, rank=2)
    base.update(kw)
    return mod.OracleCache(**base)


# ---------------------------------------------------------------- ring (Sec. 3.2/3.3/4.1)
def pin_ring_closed_form(mod):
    for W, E in [(1, 1), (2, 1), (2, 2), (3, 1), (3, 2), (3, 3), (5, 1), (5, 2), (5, 5),
                 (64, 1), (64, 2), (64, 16), (64, 64), (7, 3)]:
        c = _mk(mod, window=W, evict_chunk=E, batch=2)
        T = 4 * W + 7
        rng = np.random.default_rng(W * 100 + E)
        for t in range(T):
            k = rng.standard_normal((2, 1, 4))
            slots, ev_t, ev_s = c.append_evict(0, k, k)
            assert list(slots) == [t % W] * 2, (W, E, t)
            if t >= W and (t - W) % E == 0:
                j = (t - W) // E
                want_t = list(range(j * E, (j + 1) * E))
                want_s = [(j * E + i) % W for i in range(E)]
            else:
                want_t, want_s = [], []
            for b in range(2):
                assert ev_t[b] == want_t and ev_s[b] == want_s, (W, E, t)
            head, count, n_app = c.ring(0)
            want_count = t + 1 if t < W else W - E + 1 + ((t - W) % E)
            assert list(count) == [want_count] * 2 and list(n_app) == [t + 1] * 2
            assert count.max() <= W
            oldest = (t + 1) - want_count          # oldest live token index
            assert list(head) == [oldest % W] * 2


def pin_ring_vs_list_model(mod):
    """Naive model: python list of (token, slot); free slots kept sorted by release time."""
    rng = np.random.default_rng(0)
    for W, E in [(1, 1), (2, 1), (3, 2), (5, 3), (6, 6), (9, 4)]:
        c = _mk(mod, window=W, evict_chunk=E, batch=3)
        live = [[] for _ in range(3)]
        free = [list(range(W)) for _ in range(3)]
        ntok = [0, 0, 0]
        for step in range(6 * W + 5):
            act = rng.random(3) < 0.7
            k = rng.standard_normal((3, 1, 4))
            slots, ev_t, ev_s = c.append_evict(0, k, 2 * k, active=act)
            for b in range(3):
                if not act[b]:
                    assert slots[b] == -1 and ev_t[b] == [] and ev_s[b] == []
                    continue
                gone = []
                if len(live[b]) == W:
                    gone, live[b] = live[b][:E], live[b][E:]
                    free[b] += [s for _, s in gone]
                s = free[b].pop(0)
                live[b].append((ntok[b], s))
                ntok[b] += 1
                assert slots[b] == s
                assert ev_t[b] == [t for t, _ in gone] and ev_s[b] == [s_ for _, s_ in gone]
                # stored values are the ones appended
                seq = c.seqs[0][b]
                assert np.array_equal(seq.K[s], k[b]) and np.array_equal(seq.V[s], 2 * k[b])
                assert list(seq.live) == [t for t, _ in live[b]]


# ---------------------------------------------------------------- attention (Sec. 3.1)
def _sdpa_last_row(q, K, V, g):
    """Library routine: torch SDPA in float64; q [Hq,D], K/V [n,Hkv,D] -> [Hq,D]."""
    qt = torch.from_numpy(np.asarray(q, np.float64))[None, :, None, :]            # [1,Hq,1,D]
    Kt = torch.from_numpy(np.asarray(K, np.float64)).permute(1, 0, 2)[None]          # [1,Hkv,n,D]
    Vt = torch.from_numpy(np.asarray(V, np.float64)).permute(1, 0, 2)[None]
    Kt = Kt.repeat_interleave(g, dim=1)
    Vt = Vt.repeat_interleave(g, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt)
    return o[0, :, 0, :].numpy()


def pin_attention_full_window_is_causal(mod):
    """W >= T: every step equals full causal attention over the whole history."""
    rng = np.random.default_rng(1)
    Hq, Hkv, D, T = 6, 2, 8, 12
    c = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=T + 3)
    q = rng.standard_normal((T, 1, Hq, D))
    k = rng.standard_normal((T, 1, Hkv, D))
    v = rng.standard_normal((T, 1, Hkv, D))
    outs = []
    for t in range(T):
        o, lse, _ = c.decode_step(0, q[t], k[t], v[t])
        outs.append(o[0])
    # whole-sequence causal SDPA in one library call
    qt = torch.from_numpy(q[:, 0]).permute(1, 0, 2)[None]
    kt = torch.from_numpy(k[:, 0]).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    vt = torch.from_numpy(v[:, 0]).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True)[0]
    ref = ref.permute(1, 0, 2).numpy()
    np.testing.assert_allclose(np.stack(outs), ref, rtol=0, atol=1e-12)


def pin_attention_sliding_window(mod):
    """T > W, E = 1: step t sees exactly tokens (t-W, t]."""
    rng = np.random.default_rng(2)
    Hq, Hkv, D, W, T = 4, 2, 8, 5, 17
    c = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W)
    q = rng.standard_normal((T, 1, Hq, D))
    k = rng.standard_normal((T, 1, Hkv, D))
    v = rng.standard_normal((T, 1, Hkv, D))
    for t in range(T):
        o, _, _ = c.decode_step(0, q[t], k[t], v[t])
        lo = max(0, t - W + 1)
        ref = _sdpa_last_row(q[t, 0], k[lo:t + 1, 0], v[lo:t + 1, 0], Hq // Hkv)
        np.testing.assert_allclose(o[0], ref, rtol=0, atol=1e-12)


def pin_attention_chunked_window(mod):
    """E > 1: the live set after step t is tokens [t+1-count(t), t]."""
    rng = np.random.default_rng(3)
    Hq, Hkv, D, W, E, T = 2, 1, 4, 8, 3, 30
    c = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W, evict_chunk=E)
    q = rng.standard_normal((T, 1, Hq, D))
    k = rng.standard_normal((T, 1, Hkv, D))
    v = rng.standard_normal((T, 1, Hkv, D))
    for t in range(T):
        o, _, _ = c.decode_step(0, q[t], k[t], v[t])
        count = t + 1 if t < W else W - E + 1 + ((t - W) % E)
        lo = t + 1 - count
        ref = _sdpa_last_row(q[t, 0], k[lo:t + 1, 0], v[lo:t + 1, 0], 2)
        np.testing.assert_allclose(o[0], ref, rtol=0, atol=1e-12)


def pin_attention_window_one(mod):
    rng = np.random.default_rng(4)
    c = _mk(mod, n_q_heads=4, n_kv_heads=2, head_dim=4, window=1)
    for t in range(5):
        q = rng.standard_normal((1, 4, 4))
        k = rng.standard_normal((1, 2, 4))
        v = rng.standard_normal((1, 2, 4))
        o, lse, _ = c.decode_step(0, q, k, v)
        want = np.repeat(v[0], 2, axis=0)       # head h reads kv head h // 2
        assert np.array_equal(o[0], want)


def pin_attention_special_cases(mod):
    rng = np.random.default_rng(5)
    n, D = 9, 6
    q = rng.standard_normal(D)
    V = rng.standard_normal((n, D))
    # all keys equal -> mean of V, lse = s + log n
    K = np.tile(rng.standard_normal(D), (n, 1))
    o, lse = mod.attention_one_head(q, K, V)
    np.testing.assert_allclose(o, V.mean(0), atol=1e-13)
    np.testing.assert_allclose(lse, K[0] @ q / np.sqrt(D) + np.log(n), atol=1e-12)
    # one dominant key -> its value
    K = rng.standard_normal((n, D)) * 0.01
    K[3] = q * 1e4 / (q @ q)
    o, _ = mod.attention_one_head(q, K, V)
    np.testing.assert_allclose(o, V[3], atol=1e-12)
    # two keys, logits differing by log 3 -> weights 3/4, 1/4 (checks the 1/sqrt(d) scale)
    D2 = 4
    q2 = np.array([2.0, 0, 0, 0])
    K2 = np.array([[np.log(3.0), 0, 0, 0], [0.0, 0, 0, 0]])       # s = 2*log3/sqrt(4) = log 3
    V2 = np.array([[1.0, 0, 0, 0], [0.0, 1, 0, 0]])
    o2, lse2 = mod.attention_one_head(q2, K2, V2)
    np.testing.assert_allclose(o2, [0.75, 0.25, 0, 0], atol=1e-14)
    np.testing.assert_allclose(lse2, np.log(4.0), atol=1e-14)
    # permutation of cache order leaves o unchanged; lse equals scipy's logsumexp
    from scipy.special import logsumexp
    K = rng.standard_normal((n, D))
    o_a, lse_a = mod.attention_one_head(q, K, V)
    perm = rng.permutation(n)
    o_b, lse_b = mod.attention_one_head(q, K[perm], V[perm])
    np.testing.assert_allclose(o_a, o_b, atol=1e-14)
    np.testing.assert_allclose(lse_a, logsumexp(K @ q / np.sqrt(D)), atol=1e-13)
    # large logits do not overflow
    o_c, lse_c = mod.attention_one_head(q * 1e3, K * 1e3, V)
    assert np.all(np.isfinite(o_c)) and np.isfinite(lse_c)


def pin_attention_gqa_mapping(mod):
    rng = np.random.default_rng(6)
    for Hq, Hkv in [(4, 1), (7, 7), (8, 2), (28, 4), (6, 3)]:
        D, n = 8, 11
        q = rng.standard_normal((Hq, D))
        K = rng.standard_normal((n, Hkv, D))
        V = rng.standard_normal((n, Hkv, D))
        o, _ = mod.attention_gqa(q, K, V)
        np.testing.assert_allclose(o, _sdpa_last_row(q, K, V, Hq // Hkv), atol=1e-12)


# ---------------------------------------------------------------- encoder (Sec. 3.3, Eq. 3)
def _frac_mat(a):
    return [[Fraction(int(x)) for x in row] for row in a]


def _fmatmul(A, B):
    return [[sum(A[i][k] * B[k][j] for k in range(len(B))) for j in range(len(B[0]))] for i in range(len(A))]


def _ft(A):
    return [list(r) for r in zip(*A)]


def _exact_state(Wq, qg, Wk, Wv, Ke, Ve):
    """Eq. (3) in exact rational arithmetic, element loops only."""
    Qa = _fmatmul(_frac_mat(qg), _ft(_frac_mat(Wq)))
    Ka = _fmatmul(_frac_mat(Ke), _ft(_frac_mat(Wk)))
    Va = _fmatmul(_frac_mat(Ve), _ft(_frac_mat(Wv)))
    P = _fmatmul(Qa, _ft(Ka))
    return Qa, _fmatmul(P, Va)


def _read_golden(name):
    out = {}
    with open(os.path.join(HERE, "golden", name)) as f:
        for line in f:
            if line.startswith("#") or ":" not in line:
                continue
            head, vals = line.split(":")
            nm, r, c = head.split()
            out[nm] = np.array([float(x) for x in vals.split()]).reshape(int(r), int(c))
    return out


def pin_encode_worked_example(mod):
    g = _read_golden("encode_worked_example.txt")
    Qa = mod.latent_queries(g["Wq_a"], g["q_g"])
    assert np.array_equal(Qa, g["Q_a"])
    S1 = mod.context_state(Qa, g["Wk_a"], g["Wv_a"], g["K_e"], g["V_e"])
    assert np.array_equal(S1, g["S_prime"])
    # initial state uses the same form with the global tokens as the "evicted" rows
    assert np.array_equal(mod.initial_state(Qa, g["Wk_a"], g["Wv_a"], g["K_e"], g["V_e"]), g["S_prime"])
    assert np.array_equal(mod.initial_state(Qa, g["Wk_a"], g["Wv_a"], None, None), np.zeros((2, 2)))
    n0 = mod.normalize(g["S_prime"], 0)
    np.testing.assert_allclose(n0, [[8 / np.sqrt(113), -7 / np.sqrt(113)], [0, -1]], atol=1e-15)
    np.testing.assert_allclose(mod.normalize(g["S_prime"], 1), g["S_prime"] / np.sqrt(149), atol=1e-15)
    assert np.array_equal(mod.normalize(g["S_prime"], 2), g["S_prime"])
    # Normalize(S + S') with S = [[1,0],[0,1]]: rows [9,-7]/sqrt(130), [0,-5]/5
    S = mod.encode_update(np.eye(2), Qa, g["Wk_a"], g["Wv_a"], g["K_e"], g["V_e"], 0)
    np.testing.assert_allclose(S, [[9 / np.sqrt(130), -7 / np.sqrt(130)], [0, -1]], atol=1e-15)


def pin_encode_exact_rational(mod):
    """Small random integer problems, non-square in every dimension, vs exact arithmetic."""
    rng = np.random.default_rng(7)
    for G, r, dq, dkv, m in [(2, 3, 4, 5, 6), (3, 2, 5, 4, 1), (1, 1, 1, 1, 1), (4, 5, 3, 2, 7)]:
        Wq = rng.integers(-3, 4, (r, dq))
        qg = rng.integers(-3, 4, (G, dq))
        Wk = rng.integers(-3, 4, (r, dkv))
        Wv = rng.integers(-3, 4, (r, dkv))
        Ke = rng.integers(-3, 4, (m, dkv))
        Ve = rng.integers(-3, 4, (m, dkv))
        Qa_x, S_x = _exact_state(Wq, qg, Wk, Wv, Ke, Ve)
        Qa = mod.latent_queries(Wq, qg)
        S = mod.context_state(Qa, Wk, Wv, Ke, Ve)
        assert S.shape == (G, r)
        assert np.array_equal(Qa, np.array(Qa_x, dtype=np.float64))
        assert np.array_equal(S, np.array(S_x, dtype=np.float64))


def pin_encode_identities(mod):
    rng = np.random.default_rng(8)
    G, r, dkv, m = 5, 3, 7, 6
    Qa = rng.standard_normal((G, r))
    Wk = rng.standard_normal((r, dkv))
    Wv = rng.standard_normal((r, dkv))
    Ke = rng.standard_normal((m, dkv))
    Ve = rng.standard_normal((m, dkv))
    S1 = mod.context_state(Qa, Wk, Wv, Ke, Ve)
    # linear in the evicted set: a chunk equals the sum of its single-token states
    parts = sum(mod.context_state(Qa, Wk, Wv, Ke[i:i + 1], Ve[i:i + 1]) for i in range(m))
    np.testing.assert_allclose(S1, parts, atol=1e-12)
    # order of the evicted tokens inside a chunk does not matter
    p = rng.permutation(m)
    np.testing.assert_allclose(S1, mod.context_state(Qa, Wk, Wv, Ke[p], Ve[p]), atol=1e-12)
    # associativity (Q K^T) V = Q (K^T V), and the rank-1 form sum_i (Q_a k_a,i) v_a,i^T
    Ka, Va = Ke @ Wk.T, Ve @ Wv.T
    np.testing.assert_allclose(S1, Qa @ (Ka.T @ Va), atol=1e-12)
    np.testing.assert_allclose(S1, np.einsum("gr,ir,is->gs", Qa, Ka, Va), atol=1e-12)
    # bilinear: scaling keys by a and values by b scales S' by a*b; no softmax, no 1/sqrt(r)
    np.testing.assert_allclose(mod.context_state(Qa, Wk, Wv, 3 * Ke, -2 * Ve), -6 * S1, atol=1e-11)
    # normalize invariants
    X = rng.standard_normal((G, r))
    N0 = mod.normalize(X, 0)
    np.testing.assert_allclose(np.linalg.norm(N0, axis=1), 1.0, atol=1e-14)
    np.testing.assert_allclose(mod.normalize(7.5 * X, 0), N0, atol=1e-14)
    np.testing.assert_allclose(np.linalg.norm(mod.normalize(X, 1)), 1.0, atol=1e-14)
    np.testing.assert_allclose(mod.normalize(0.01 * X, 1), mod.normalize(X, 1), atol=1e-14)
    assert np.array_equal(mod.normalize(np.zeros((2, 3)), 0), np.zeros((2, 3)))   # no 0/0


def pin_encode_recurrence(mod):
    """State through a rollout: fixed size, Global-Only, #Global-0, constant-token fixed point."""
    rng = np.random.default_rng(9)
    Hq, Hkv, D, W, G, r = 4, 2, 4, 3, 3, 2
    dq, dkv = Hq * D, Hkv * D
    P = dict(Wq_a=rng.standard_normal((r, dq)), Wk_a=rng.standard_normal((r, dkv)),
             Wv_a=rng.standard_normal((r, dkv)), q_g=rng.standard_normal((G, dq)),
             k_g=rng.standard_normal((G, dkv)), v_g=rng.standard_normal((G, dkv)))
    T = 11
    q = rng.standard_normal((T, 1, Hq, D))
    k = rng.standard_normal((T, 1, Hkv, D))
    v = rng.standard_normal((T, 1, Hkv, D))

    def run(**kw):
        c = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, n_global=G, rank=r,
                **{"window": W, **kw.pop("cfg", {})})
        c.set_encoder(0, **{**P, **kw})
        states = [c.S[0][0].copy()]
        for t in range(T):
            c.decode_step(0, q[t], k[t], v[t])
            states.append(c.S[0][0].copy())
        return states

    # (a) E = 1, mode 0: S_{t} = Normalize(S_{t-1} + S'(token t-W)), rebuilt from the history
    st = run()
    Qa = P["q_g"] @ P["Wq_a"].T
    S = (Qa @ (P["k_g"] @ P["Wk_a"].T).T) @ (P["v_g"] @ P["Wv_a"].T)
    np.testing.assert_allclose(st[0], S, atol=1e-12)
    for t in range(T):
        if t >= W:
            e = t - W
            ka = P["Wk_a"] @ k[e, 0].reshape(-1)
            va = P["Wv_a"] @ v[e, 0].reshape(-1)
            S = S + np.outer(Qa @ ka, va)
            S = S / np.linalg.norm(S, axis=1, keepdims=True)
        np.testing.assert_allclose(st[t + 1], S, atol=1e-12)
        assert st[t + 1].shape == (G, r)                      # fixed size for any length
    # (b) Global-Only ablation and W >= T: state never moves
    for s in run(cfg=dict(encode_enabled=0)):
        assert np.array_equal(s, st[0])
    for s in run(cfg=dict(window=T)):
        assert np.array_equal(s, st[0])
    # (c) #Global-0: zero start, first update gives Normalize(S')
    st0 = run(k_g=None, v_g=None)
    assert np.array_equal(st0[0], np.zeros((G, r)))
    ka, va = P["Wk_a"] @ k[0, 0].reshape(-1), P["Wv_a"] @ v[0, 0].reshape(-1)
    S1 = np.outer(Qa @ ka, va)
    np.testing.assert_allclose(st0[W + 1], S1 / np.linalg.norm(S1, axis=1, keepdims=True), atol=1e-12)
    # (d) chunked eviction folds E tokens at once, with one Normalize per chunk
    E = 2
    stE = run(cfg=dict(evict_chunk=E))
    S = st[0].copy()
    for t in range(T):
        if t >= W and (t - W) % E == 0:
            j = (t - W) // E
            for e in range(j * E, (j + 1) * E):
                S = S + np.outer(Qa @ (P["Wk_a"] @ k[e, 0].reshape(-1)), P["Wv_a"] @ v[e, 0].reshape(-1))
            S = S / np.linalg.norm(S, axis=1, keepdims=True)
        np.testing.assert_allclose(stE[t + 1], S, atol=1e-12)
    # (e) identical tokens, zero start: the state is the fixed point Normalize(S') after every update
    c = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, n_global=G, rank=r, window=2)
    c.set_encoder(0, **{**P, "k_g": None, "v_g": None})
    for t in range(9):
        c.decode_step(0, q[t], k[0], v[0])
        if t >= 2:
            np.testing.assert_allclose(c.S[0][0], S1 / np.linalg.norm(S1, axis=1, keepdims=True), atol=1e-12)
    # (f) modes 1 and 2
    c1 = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, n_global=G, rank=r, window=W, normalize_mode=1)
    c2 = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, n_global=G, rank=r, window=W, normalize_mode=2)
    c1.set_encoder(0, **P)
    c2.set_encoder(0, **P)
    S2 = st[0].copy()
    for t in range(T):
        c1.decode_step(0, q[t], k[t], v[t])
        c2.decode_step(0, q[t], k[t], v[t])
        if t >= W:
            e = t - W
            S2 = S2 + np.outer(Qa @ (P["Wk_a"] @ k[e, 0].reshape(-1)), P["Wv_a"] @ v[e, 0].reshape(-1))
            np.testing.assert_allclose(np.linalg.norm(c1.S[0][0]), 1.0, atol=1e-13)
        np.testing.assert_allclose(c2.S[0][0], S2, atol=1e-10)


def pin_staged_rows_are_evicted_tokens(mod):
    """The rows handed to the encoder are the evicted tokens' K/V, heads concatenated, oldest first."""
    rng = np.random.default_rng(10)
    Hkv, D, W, E = 3, 2, 4, 2
    c = _mk(mod, n_q_heads=3, n_kv_heads=Hkv, head_dim=D, window=W, evict_chunk=E)
    ks = rng.standard_normal((10, 1, Hkv, D))
    vs = rng.standard_normal((10, 1, Hkv, D))
    for t in range(10):
        _, ev_t, _ = c.append_evict(0, ks[t], vs[t])
        st = c.staged[0][0]
        if ev_t[0]:
            assert np.array_equal(st[0], np.stack([ks[e, 0].reshape(-1) for e in ev_t[0]]))
            assert np.array_equal(st[1], np.stack([vs[e, 0].reshape(-1) for e in ev_t[0]]))
        else:
            assert st is None

# ---------------------------------------------------------------- pinned prompt (Sec. 3.3 policy, Sec. 4.1)
def pin_prompt_is_pinned_and_window_slides_over_the_rest(mod):
    """A prompt of n tokens keeps its n cache entries for the whole rollout, every query attends to it, only
    reasoning tokens are evicted (oldest first, at most the sliding capacity per chunk) and the cache never holds
    more than W tokens.  Slots and evictions against closed forms, attention against the library routine on the
    token set worked out from the history."""
    rng = np.random.default_rng(11)
    Hq, Hkv, D = 4, 2, 8
    for W, n, E in [(8, 3, 1), (8, 3, 2), (8, 6, 4), (8, 7, 1), (9, 1, 8), (6, 0, 2), (12, 5, 3)]:
        cap = W - n
        Ee = min(E, cap)
        T = 3 * W + 5
        c = _mk(mod, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W, evict_chunk=E, batch=2)
        Kp = rng.standard_normal((2, max(n, 1), Hkv, D))
        Vp = rng.standard_normal((2, max(n, 1), Hkv, D))
        c.prefill(0, Kp, Vp, [n, n])
        assert list(c.pinned_count(0)) == [n, n]
        hist_k = [Kp[0, i] for i in range(n)]
        hist_v = [Vp[0, i] for i in range(n)]
        for j in range(T):                                  # j-th reasoning token, global index n + j
            q = rng.standard_normal((2, Hq, D))
            k = rng.standard_normal((2, Hkv, D))
            v = rng.standard_normal((2, Hkv, D))
            o, _, (slots, ev_t, ev_s) = c.decode_step(0, q, k, v)
            hist_k.append(k[0]); hist_v.append(v[0])
            assert list(slots) == [n + j % cap] * 2, (W, n, E, j)
            if j >= cap and (j - cap) % Ee == 0:
                first = (j - cap) // Ee * Ee
                want_t = [n + first + i for i in range(Ee)]
                want_s = [n + (first + i) % cap for i in range(Ee)]
            else:
                want_t, want_s = [], []
            assert ev_t[0] == want_t and ev_s[0] == want_s, (W, n, E, j)
            assert all(t >= n for t in ev_t[0])             # a prompt token never leaves
            held = j + 1 if j < cap else cap - Ee + 1 + (j - cap) % Ee
            head, count, n_app = c.ring(0)
            assert list(count) == [held] * 2 and list(n_app) == [n + j + 1] * 2 and n + held <= W
            live = list(range(n)) + list(range(n + j + 1 - held, n + j + 1))
            ref = _sdpa_last_row(q[0], np.stack([hist_k[t] for t in live]), np.stack([hist_v[t] for t in live]),
                                 Hq // Hkv)
            np.testing.assert_allclose(o[0], ref, rtol=0, atol=1e-12)


def pin_prompt_rows_never_reach_the_encoder(mod):
    """Only evicted reasoning tokens are staged for the encoder; with no prompt the cache behaves as before."""
    rng = np.random.default_rng(12)
    Hkv, D, W, n = 2, 3, 6, 4
    c = _mk(mod, n_q_heads=2, n_kv_heads=Hkv, head_dim=D, window=W, evict_chunk=1)
    Kp = rng.standard_normal((1, n, Hkv, D))
    c.prefill(0, Kp, -Kp, [n])
    ks = rng.standard_normal((9, 1, Hkv, D))
    for j in range(9):
        _, ev_t, _ = c.append_evict(0, ks[j], 2 * ks[j])
        st = c.staged[0][0]
        if j >= W - n:
            assert ev_t[0] == [n + j - (W - n)]
            assert np.array_equal(st[0], ks[j - (W - n), 0].reshape(1, -1))
            assert np.array_equal(st[1], 2 * ks[j - (W - n), 0].reshape(1, -1))
        else:
            assert st is None and ev_t[0] == []
    a, b = _mk(mod, window=5), _mk(mod, window=5)
    b.prefill(0, np.zeros((1, 1, 1, 4)), np.zeros((1, 1, 1, 4)), [0])
    for t in range(12):
        x = rng.standard_normal((1, 1, 4))
        ra, rb = a.append_evict(0, x, x), b.append_evict(0, x, x)
        assert list(ra[0]) == list(rb[0]) and ra[1] == rb[1] and ra[2] == rb[2]

# ---------------------------------------------------------------- dynamic weight update (Sec. 3.3)
def pin_lora_update(mod):
    """Delta W = A S B on a hand-worked integer case, in exact rational arithmetic, and through the identities
    (W + Delta W) x = W x + A (S (B x)), linearity in S, S = 0 changes nothing."""
    A = np.array([[1, 2], [0, -1], [3, 1]])             # d_out 3, G 2
    S = np.array([[2, 0, 1], [-1, 1, 0]])               # G 2, r 3
    Bm = np.array([[1, 0, 2, 0], [0, 1, 0, -1], [1, 1, 0, 0]])   # r 3, d_in 4
    # S B = [[3,1,4,0],[-1,1,-2,-1]];  A (S B) = [[1,3,0,-2],[1,-1,2,1],[8,4,10,-1]]
    assert np.array_equal(mod.lora_delta(A, S, Bm), np.array([[1, 3, 0, -2], [1, -1, 2, 1], [8, 4, 10, -1]]))
    rng = np.random.default_rng(21)
    d_out, G, r, d_in, B = 5, 3, 4, 6, 2
    Ai, Si, Bi = rng.integers(-4, 5, (d_out, G)), rng.integers(-4, 5, (B, G, r)), rng.integers(-4, 5, (r, d_in))
    xi, yi = rng.integers(-4, 5, (B, d_in)), rng.integers(-4, 5, (B, d_out))
    got = mod.lora_apply(yi, xi, Ai, Si, Bi)
    for b in range(B):
        for i in range(d_out):
            want = Fraction(int(yi[b, i]))
            for g in range(G):
                for j in range(r):
                    for d in range(d_in):
                        want += Fraction(int(Ai[i, g])) * int(Si[b, g, j]) * int(Bi[j, d]) * int(xi[b, d])
            assert Fraction(float(got[b, i])) == want
    Af, Sf, Bf = rng.standard_normal((d_out, G)), rng.standard_normal((B, G, r)), rng.standard_normal((r, d_in))
    x, Wm = rng.standard_normal((B, d_in)), rng.standard_normal((d_out, d_in))
    y = x @ Wm.T
    full = np.stack([(Wm + mod.lora_delta(Af, Sf[b], Bf)) @ x[b] for b in range(B)])
    np.testing.assert_allclose(mod.lora_apply(y, x, Af, Sf, Bf), full, atol=1e-12)
    fact = np.stack([y[b] + Af @ (Sf[b] @ (Bf @ x[b])) for b in range(B)])
    np.testing.assert_allclose(mod.lora_apply(y, x, Af, Sf, Bf), fact, atol=1e-12)
    np.testing.assert_allclose(mod.lora_apply(y, x, Af, 0 * Sf, Bf), y, atol=0)
    two = mod.lora_apply(y, x, Af, 2 * Sf, Bf) - y
    np.testing.assert_allclose(two, 2 * (mod.lora_apply(y, x, Af, Sf, Bf) - y), atol=1e-12)

def pin_reset_gives_a_fresh_sequence(mod):
    """After a reset a sequence behaves exactly like one in a new cache (same slots, evictions, outputs, state),
    and the sequences that were not reset are untouched."""
    rng = np.random.default_rng(31)
    kw = dict(n_q_heads=2, n_kv_heads=1, head_dim=4, window=5, evict_chunk=2, batch=2, n_global=3, rank=2)
    a, fresh = _mk(mod, **kw), _mk(mod, **kw)
    enc = dict(Wq_a=rng.standard_normal((2, 8)), Wk_a=rng.standard_normal((2, 4)), Wv_a=rng.standard_normal((2, 4)),
               q_g=rng.standard_normal((3, 8)), k_g=rng.standard_normal((3, 4)), v_g=rng.standard_normal((3, 4)))
    a.set_encoder(0, **enc)
    fresh.set_encoder(0, **enc)
    for t in range(9):
        x = rng.standard_normal((2, 1, 4))
        a.decode_step(0, rng.standard_normal((2, 2, 4)), x, x)
    kept_S, kept_ring = a.S[0][1].copy(), [r[1] for r in a.ring(0)]
    a.reset([1, 0])
    assert [r[1] for r in a.ring(0)] == kept_ring and np.array_equal(a.S[0][1], kept_S)
    assert [r[0] for r in a.ring(0)] == [0, 0, 0] and list(a.pinned_count(0)) == [0, 0]
    for t in range(9):
        q, x = rng.standard_normal((2, 2, 4)), rng.standard_normal((2, 1, 4))
        oa, _, ra = a.decode_step(0, q, x, x, active=[1, 0])
        of, _, rf = fresh.decode_step(0, q, x, x, active=[1, 0])
        assert np.array_equal(oa[0], of[0]) and ra[0][0] == rf[0][0] and ra[1][0] == rf[1][0]
        assert np.array_equal(a.S[0][0], fresh.S[0][0])


# ---------------------------------------------------------------- importance-aware eviction (Sec. 4.3 token dropping)
def _score_cfg(mod, W, E, recent, **kw):
    return _mk(mod, window=W, evict_chunk=E, policy="score", recent=recent, **kw)


def pin_score_hand_worked(mod):
    """Hq = Hkv = 1, D = 1, all queries zero, so every softmax is uniform and the masses are dyadic fractions.
    W = 2, E = 1, nothing protected: token 0 collects 1, then 1/2 per step; every later token has 1/2 when the next
    one arrives and is the one that leaves -- from its slot 1, which the newcomer takes.  With the newest token
    protected the only candidate is the oldest: plain FIFO."""
    c = _score_cfg(mod, 2, 1, 0, n_q_heads=1, n_kv_heads=1, head_dim=1, batch=1)
    q0 = np.zeros((1, 1, 1))
    left, slots = [], []
    for t in range(6):
        x = np.full((1, 1, 1), float(t + 1))
        _, _, (sl, ev_t, ev_s) = c.decode_step(0, q0, x, x)
        left.append(ev_t[0]); slots.append(int(sl[0]))
    assert left == [[], [], [1], [2], [3], [4]] and slots == [0, 1, 1, 1, 1, 1]
    assert c.scores(0, 0) == {0: 1.0 + 5 * 0.5, 5: 0.5}
    assert c.margin[0][0] == (1.0 + 4 * 0.5) - 0.5              # token 0 stayed with 3.0 when token 4 left with 0.5
    f = _score_cfg(mod, 2, 1, 1, n_q_heads=1, n_kv_heads=1, head_dim=1, batch=1)
    left = []
    for t in range(6):
        x = np.full((1, 1, 1), float(t + 1))
        left.append(f.decode_step(0, q0, x, x)[2][1][0])
    assert left == [[], [], [0], [1], [2], [3]]


def _naive_score_rollout(W, E, recent, n_prompt, q, kk, vv, Hq, Hkv):
    """Independent model.  Rows of kk, vv are the tokens in arrival order, the first n_prompt of them a pinned
    prompt.  The whole history is kept; the scores at an eviction are recomputed from scratch as the sum, over every
    earlier step, of the torch softmax weights that step's query gave the token."""
    g = Hq // Hkv
    T, D = q.shape[0], q.shape[-1]
    live = list(range(n_prompt))
    attn_hist, evicted_hist, live_hist, out_hist, score_hist = [], [], [], [], []
    for t in range(T):
        tok = n_prompt + t
        sliding = [x for x in live if x >= n_prompt]
        cap = W - n_prompt
        ev = []
        if len(sliding) == cap:
            m = min(E, cap)
            prot = min(recent, cap - m)
            cand = sorted(sliding)[:cap - prot]
            sc = np.array([sum(mass[lst.index(x)] for lst, mass in attn_hist if x in lst) for x in cand])
            order = np.lexsort((np.array(cand), sc))          # by score, then by token index
            ev = sorted(cand[i] for i in order[:m])
            live = [x for x in live if x not in ev]
        live.append(tok)
        K = torch.tensor(np.stack([kk[x] for x in live]))     # [n, Hkv, D]
        V = torch.tensor(np.stack([vv[x] for x in live]))
        mass = np.zeros(len(live))
        o = np.zeros((Hq, D))
        for h in range(Hq):
            w = torch.softmax(K[:, h // g] @ torch.tensor(q[t, h]) / np.sqrt(D), dim=0)
            mass += w.numpy()
            o[h] = (w @ V[:, h // g]).numpy()
        attn_hist.append((list(live), mass))
        evicted_hist.append(ev); live_hist.append(list(live)); out_hist.append(o)
        score_hist.append({x: sum(ms[lst.index(x)] for lst, ms in attn_hist if x in lst) for x in live if x >= n_prompt})
    return evicted_hist, live_hist, out_hist, score_hist


def pin_score_policy_vs_brute_force(mod):
    rng = np.random.default_rng(77)
    Hq, Hkv, D = 4, 2, 4
    for W, E, recent, n_prompt in [(4, 1, 0, 0), (6, 2, 1, 0), (9, 3, 3, 2), (5, 5, 0, 0), (7, 2, 4, 3), (6, 1, 5, 0)]:
        T = 40
        q = rng.standard_normal((T, Hq, D)) * 2
        k = rng.standard_normal((T, Hkv, D))
        v = rng.standard_normal((T, Hkv, D))
        kp = rng.standard_normal((n_prompt, Hkv, D))
        vp = rng.standard_normal((n_prompt, Hkv, D))
        c = _score_cfg(mod, W, E, recent, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
        if n_prompt:
            c.prefill(0, kp[None], vp[None], [n_prompt])
        ev_want, live_want, out_want, score_want = _naive_score_rollout(
            W, E, recent, n_prompt, q, np.concatenate([kp, k]), np.concatenate([vp, v]), Hq, Hkv)
        n_ev = 0
        for t in range(T):
            o, _, (sl, ev_t, ev_s) = c.decode_step(0, q[t][None], k[t][None], v[t][None])
            assert ev_t[0] == ev_want[t], (W, E, recent, n_prompt, t, ev_t[0], ev_want[t])
            assert sorted(list(c.seqs[0][0].pinned) + list(c.seqs[0][0].live)) == sorted(live_want[t])
            np.testing.assert_allclose(o[0], out_want[t], atol=1e-12)
            got = c.scores(0, 0)
            assert set(got) == set(score_want[t])
            for tok, val in score_want[t].items():
                assert abs(got[tok] - val) < 1e-12, (W, E, recent, n_prompt, t, tok)
            assert len(c.seqs[0][0].live) + n_prompt <= W
            n_ev += len(ev_t[0])
        assert n_ev >= T - W - 1
        # not the sliding window: some token outlived W later arrivals (except where everything is protected)
        if recent < W - n_prompt - min(E, W - n_prompt):
            assert min(c.seqs[0][0].live) < n_prompt + T - W


def pin_score_policy_reduces_to_fifo(mod):
    """(a) No attention is ever run, so every score is zero and every tie goes to the older token: the sliding window.
    (b) Everything but the E oldest tokens is protected: the candidates are exactly the tokens FIFO evicts, whatever
    the scores, and outputs, slots and states equal the sliding-window cache's."""
    rng = np.random.default_rng(5)
    for W, E in [(3, 1), (6, 2), (8, 8), (7, 3)]:
        a = _score_cfg(mod, W, E, 0, batch=2)
        f = _mk(mod, window=W, evict_chunk=E, batch=2)
        for t in range(4 * W + 3):
            x = rng.standard_normal((2, 1, 4))
            ra, rf = a.append_evict(0, x, x), f.append_evict(0, x, x)
            assert list(ra[0]) == list(rf[0]) and ra[1] == rf[1] and ra[2] == rf[2], (W, E, t)
        enc = dict(Wq_a=rng.standard_normal((2, 8)), Wk_a=rng.standard_normal((2, 4)), Wv_a=rng.standard_normal((2, 4)),
                   q_g=rng.standard_normal((3, 8)), k_g=rng.standard_normal((3, 4)), v_g=rng.standard_normal((3, 4)))
        b = _score_cfg(mod, W, E, W - E, batch=2)
        f = _mk(mod, window=W, evict_chunk=E, batch=2)
        b.set_encoder(0, **enc); f.set_encoder(0, **enc)
        for t in range(4 * W + 3):
            q, x, y = rng.standard_normal((2, 2, 4)), rng.standard_normal((2, 1, 4)), rng.standard_normal((2, 1, 4))
            ob, lb_, rb = b.decode_step(0, q, x, y)
            of, lf_, rf = f.decode_step(0, q, x, y)
            assert list(rb[0]) == list(rf[0]) and rb[1] == rf[1] and rb[2] == rf[2]
            assert np.array_equal(ob, of) and np.array_equal(b.S[0], f.S[0])


def pin_score_mass_bookkeeping(mod):
    """Every decoded token hands out exactly Hq units of mass; what the live tokens hold plus what evicted tokens took
    with them is Hq per step (no prompt).  Repeating the attention call changes nothing.  A token that draws almost
    all the attention of every step is never evicted, while the sliding window drops it after W steps."""
    rng = np.random.default_rng(9)
    Hq, Hkv, D, W, E = 4, 2, 4, 5, 2
    c = _score_cfg(mod, W, E, 1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    d = _score_cfg(mod, W, E, 1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    carried = 0.0
    for t in range(30):
        q, x = rng.standard_normal((1, Hq, D)), rng.standard_normal((1, Hkv, D))
        before = c.scores(0, 0)
        _, _, (sl, ev_t, ev_s) = c.decode_step(0, q, x, x)
        carried += sum(before[tok] for tok in ev_t[0])
        assert abs(sum(c.scores(0, 0).values()) + carried - Hq * (t + 1)) < 1e-9
        assert set(c.scores(0, 0)) == set(c.seqs[0][0].live)
        _, _, rec = d.decode_step(0, q, x, x)
        d.decode_attn(0, q); d.decode_attn(0, rng.standard_normal((1, Hq, D))); d.decode_attn(0, q)
        assert rec[1] == ev_t
    assert c.scores(0, 0) == d.scores(0, 0)
    total = sum(c.scores(0, 0).values())
    for _ in range(3):                          # tokens arriving with no attention in between: nothing is added twice
        before = c.scores(0, 0)
        _, ev_t, _ = c.append_evict(0, x, x)
        total -= sum(before[tok] for tok in ev_t[0])
        assert abs(sum(c.scores(0, 0).values()) - total) < 1e-9
    big = np.zeros((1, Hkv, D)); big[:, :, 0] = 8.0
    s = _score_cfg(mod, 4, 1, 0, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    f = _mk(mod, window=4, evict_chunk=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    qq = np.zeros((1, Hq, D)); qq[:, :, 0] = 8.0
    for t in range(40):
        x = big if t == 0 else rng.standard_normal((1, Hkv, D)) * 0.1
        s.decode_step(0, qq, x, x); f.decode_step(0, qq, x, x)
        assert 0 in s.seqs[0][0].live
    assert 0 not in f.seqs[0][0].live
    assert s.scores(0, 0)[0] > 0.99 * Hq * 40


PINS = [pin_score_hand_worked, pin_score_policy_vs_brute_force, pin_score_policy_reduces_to_fifo,
        pin_score_mass_bookkeeping, pin_ring_closed_form, pin_ring_vs_list_model, pin_attention_full_window_is_causal,
        pin_attention_sliding_window, pin_attention_chunked_window, pin_attention_window_one,
        pin_attention_special_cases, pin_attention_gqa_mapping, pin_encode_worked_example,
        pin_encode_exact_rational, pin_encode_identities, pin_encode_recurrence,
        pin_staged_rows_are_evicted_tokens, pin_prompt_is_pinned_and_window_slides_over_the_rest,
        pin_prompt_rows_never_reach_the_encoder, pin_lora_update, pin_reset_gives_a_fresh_sequence]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(O)


# =====================================================================================
# planted mistakes: each plausible slip in the oracle must trip at least one pin
# =====================================================================================
def _mutant(src_edit):
    path = O.__file__
    src = open(path).read()
    old, new = src_edit
    assert src.count(old) >= 1, old
    m = types.ModuleType("oracle_mutant")
    m.__file__ = path
    exec(compile(src.replace(old, new, 1), path, "exec"), m.__dict__)
    return m


MUTATIONS = {
    "drop_sqrt_d": ("s = (K @ q) / np.sqrt(F64(d))", "s = (K @ q)"),
    "scale_by_d": ("s = (K @ q) / np.sqrt(F64(d))", "s = (K @ q) / F64(d)"),
    "gqa_modulo": ("K[:, h // g, :], V[:, h // g, :]", "K[:, h % Hkv, :], V[:, h % Hkv, :]"),
    "swap_wk_wv": ("Ka = np.asarray(K_e, F64) @ np.asarray(Wk_a, F64).T",
                   "Ka = np.asarray(K_e, F64) @ np.asarray(Wv_a, F64).T"),
    "values_through_wk": ("Va = np.asarray(V_e, F64) @ np.asarray(Wv_a, F64).T",
                          "Va = np.asarray(V_e, F64) @ np.asarray(Wk_a, F64).T"),
    "keys_as_values": ("Va = np.asarray(V_e, F64) @", "Va = np.asarray(K_e, F64) @"),
    "encoder_softmax_scale": ("P = np.asarray(Qa, F64) @ Ka.T ", "P = np.asarray(Qa, F64) @ Ka.T / np.sqrt(Ka.shape[1]) "),
    "drop_accumulate": ("normalize(np.asarray(S, F64) + context_state(", "normalize(context_state("),
    "normalize_axis": ("n = np.sqrt(np.sum(S * S, axis=-1, keepdims=True))", "n = np.sqrt(np.sum(S * S, axis=0, keepdims=True))"),
    "evict_after_append": ("if len(c.live) == capacity:", "if len(c.live) > capacity:"),
    "evict_one_too_early": ("if len(c.live) == capacity:", "if len(c.live) == capacity - 1 and capacity > 1:"),
    "lifo_free_slots": ("s_new = c.free.popleft()", "s_new = c.free.pop()"),
    "evict_newest": ("t_old = c.live.popleft()", "t_old = c.live.pop()"),
    "new_token_not_attended": ("+ [c.slot_of[t] for t in c.live]", "+ ([c.slot_of[t] for t in list(c.live)[:-1]] or [c.slot_of[c.live[-1]]])"),
    "prompt_not_attended": ("sl = [c.slot_of[t] for t in c.pinned] + ", "sl = "),
    "prompt_gets_evicted": ("capacity = self.W - len(c.pinned)", "capacity = self.W - len(c.pinned); c.live.extendleft(reversed(c.pinned)); c.pinned = []"),
    "window_ignores_prompt": ("capacity = self.W - len(c.pinned) ", "capacity = self.W "),
    "chunk_exceeds_capacity": ("for _ in range(min(self.E, capacity)):", "for _ in range(self.E):"),
    "stale_v": ("c.V[s_new] = v_new[b]", "c.V[s_new] = k_new[b]"),
    "encode_ignores_disable": ("if not self.encode_enabled:\n            return", "if False:\n            return"),
    "lora_transposed_state": ("return np.asarray(A, F64) @ np.asarray(S, F64) @ np.asarray(Bm, F64)",
                              "return np.asarray(A, F64) @ np.asarray(S, F64).T @ np.asarray(Bm, F64)"),
    "lora_replaces_output": ("y[b] = y[b] + lora_delta(A, S[b], Bm) @ x[b]", "y[b] = lora_delta(A, S[b], Bm) @ x[b]"),
    "lora_shared_state": ("y[b] = y[b] + lora_delta(A, S[b], Bm) @ x[b]", "y[b] = y[b] + lora_delta(A, S[0], Bm) @ x[b]"),
    "lse_without_max": ("return o, smax + np.log(z)", "return o, np.log(z)"),
    "score_ties_to_newer": ("key=lambda tok: (c.score[tok], tok))[:m]", "key=lambda tok: (c.score[tok], -tok))[:m]"),
    "score_evicts_highest": ("key=lambda tok: (c.score[tok], tok))[:m]", "key=lambda tok: (-c.score[tok], tok))[:m]"),
    "score_ignores_recent": ("protected = min(self.recent, capacity - m)", "protected = 0"),
    "score_protection_blocks_eviction": ("protected = min(self.recent, capacity - m)", "protected = min(self.recent, capacity - 1)"),
    "score_first_head_only": ("    for h in range(Hq):\n        s = (K[:, h // g, :] @ q[h]) / np.sqrt(F64(D))",
                              "    for h in range(1):\n        s = (K[:, h // g, :] @ q[h]) / np.sqrt(F64(D))"),
    "score_unnormalised_mass": ("        mass += e / np.sum(e)", "        mass += e"),
    "score_mass_without_scale": ("s = (K[:, h // g, :] @ q[h]) / np.sqrt(F64(D))\n        e = np.exp(s - np.max(s))\n        mass",
                                 "s = (K[:, h // g, :] @ q[h])\n        e = np.exp(s - np.max(s))\n        mass"),
    "score_leave_in_score_order": ("for t_old in sorted(chosen):", "for t_old in chosen:"),
    "score_folded_twice": ("                    c.score[t_tok] += m_tok\n                c.pending = None",
                           "                    c.score[t_tok] += m_tok"),
    "score_new_token_gets_no_mass": ("c.pending = (list(c.live), mass[len(c.pinned):])",
                                     "c.pending = (list(c.live)[:-1], mass[len(c.pinned):-1])"),
    "score_pinned_offset_forgotten": ("c.pending = (list(c.live), mass[len(c.pinned):])",
                                      "c.pending = (list(c.live), mass[:len(c.live)])"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name):
    m = _mutant(MUTATIONS[name])
    caught = []
    for pin in PINS:
        try:
            pin(m)
        except Exception:   # assertion or shape error: either way the pin trips
            caught.append(pin.__name__)
    assert caught, f"no pin detects mutation {name}"
