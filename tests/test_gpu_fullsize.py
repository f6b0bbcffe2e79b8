"""GPU parity at the full sizes of the five configurations, in the launch mode the benchmark times
(ptenc_decode_step with layer = -1), on outputs the oracle can compute one by one.

Two kinds of run:
* full L, B, W: the rings are filled from the synthetic stream, then a stretch of steady-state steps runs; attention
  outputs and encoder states are checked at sampled (layer, sequence, step) points that include the first step, the
  last step before the ring is full, the first evictions and the wrap of the ring;
* whole rollouts (every one of the T steps, ragged lengths for the Llama-shaped workload) with two layers: slot
  indices and eviction order of every step and sequence are compared bit for bit, outputs and states at samples.

The oracle side regenerates the tokens of one (layer, sequence) by random access and keeps its own explicit
deque/free-list cache; nothing it uses comes from the CUDA path.
"""
import numpy as np
import pytest
import torch

import paper_2602_16839_b200 as pt
from oracle.ptenc_oracle import (OracleCache, attention_gqa, encode_update, initial_state, latent_queries)
from ptenc_inputs import CONFIGS, make_inputs, stress_config

from _harness import TOL_OUT, TOL_STATE, np64

pytestmark = pytest.mark.gpu


def _workload(name):
    if name.startswith("stress"):
        _, w, b = name.split("-")
        c = stress_config(int(w[1:]), int(b[1:]))
    else:
        c = dict(CONFIGS[name])
    return c


class _IntOracle:
    """The oracle's explicit cache bookkeeping for a few sampled sequences (payload one number per token)."""

    def __init__(self, seqs, W, E):
        self.seqs = list(seqs)
        self.o = OracleCache(n_layers=1, batch=len(self.seqs), n_q_heads=1, n_kv_heads=1, head_dim=1, window=W,
                             evict_chunk=E, n_global=1, rank=1)
        self.evicted = [[] for _ in self.seqs]           # token indices in eviction order

    def prefill(self, n_prompt_all):
        n = [int(n_prompt_all[b]) for b in self.seqs]
        z = np.zeros((len(self.seqs), max(max(n), 1), 1, 1))
        self.o.prefill(0, z, z, n)

    def pinned(self, i):
        return list(self.o.seqs[0][i].pinned)

    def step(self, active_all):
        act = None if active_all is None else [int(active_all[b]) for b in self.seqs]
        z = np.zeros((len(self.seqs), 1, 1))
        slots, ev_t, ev_s = self.o.append_evict(0, z, z, act)
        for i, toks in enumerate(ev_t):
            self.evicted[i].extend(toks)
        return slots, ev_t, ev_s

    def live(self, i):
        return list(self.o.seqs[0][i].live)


def _oracle_out(gen, layer, b, t_query, live_tokens):
    K, V = gen.token_kv(layer, b, live_tokens)
    q = gen.token_q(layer, b, t_query)
    o, _ = attention_gqa(np64(q), np64(K), np64(V))
    return o


def _oracle_state(gen, layer, b, evicted_chunks, mode=0):
    """State of (layer, b) after folding the given chunks of evicted tokens, in order."""
    P = {k: np64(v) for k, v in gen.encoder_params(layer, device="cpu").items()}
    Qa = latent_queries(P["Wq_a"], P["q_g"])
    S = initial_state(Qa, P["Wk_a"], P["Wv_a"], P["k_g"], P["v_g"])
    flat = [tok for toks in evicted_chunks for tok in toks]
    Ks, Vs = [], []
    for lo in range(0, len(flat), 4096):                      # regenerate the evicted tokens' rows in batches
        K, V = gen.token_kv(layer, b, flat[lo:lo + 4096])
        Ks.append(np64(K).reshape(K.shape[0], -1))
        Vs.append(np64(V).reshape(V.shape[0], -1))
    if not flat:
        return S
    K, V = np.concatenate(Ks), np.concatenate(Vs)
    at = 0
    for toks in evicted_chunks:
        if toks:
            S = encode_update(S, Qa, P["Wk_a"], P["Wv_a"], K[at:at + len(toks)], V[at:at + len(toks)], mode)
            at += len(toks)
    return S


def _make_cache(c, L, dev="cuda:0", evict_chunk=1):
    gen = make_inputs({**c, "n_layers": L}, seed=0, device=dev)
    cfg = pt.make_config(n_layers=L, batch=c["batch"], n_q_heads=c["n_q_heads"], n_kv_heads=c["n_kv_heads"],
                         head_dim=c["head_dim"], window=c["window"], evict_chunk=evict_chunk,
                         n_global=c["n_global"], rank=c["rank"], dtype=c["dtype"])
    cache = pt.Cache(cfg)
    for l in range(L):
        P = gen.encoder_params(l)
        cache.set_encoder(l, P["Wq_a"], P["Wk_a"], P["Wv_a"], P["q_g"], P["k_g"], P["v_g"])
    return gen, cache


@pytest.mark.parametrize("name,steady", [("qwen3b", 40), ("qwen7b", 40), ("llama8b", 24), ("stress-w512-b16", 600),
                                         ("stress-w4096-b256", 12)])
def test_full_size_benchmark_launch_mode(name, steady):
    c = _workload(name)
    L, B, W, Hq, D = c["n_layers"], c["batch"], c["window"], c["n_q_heads"], c["head_dim"]
    torch.cuda.empty_cache()
    gen, cache = _make_cache(c, L)
    assert cache.info()["tensor_core_attn"]
    rng = np.random.default_rng(1234)
    seqs = sorted({0, B - 1, *rng.integers(0, B, 4).tolist()})
    layers = sorted({0, L - 1, *rng.integers(0, L, 3).tolist()})
    io = _IntOracle(seqs, W, 1)
    T = W + steady
    check_steps = {0, 1, W // 2, W - 2, W - 1, W, W + 1, W + 2, T - 1}
    if T > 2 * W:
        check_steps |= {2 * W - 1, 2 * W, 2 * W + 1}
    check_steps |= set(rng.integers(W, T, 6).tolist())
    out = torch.zeros(L, B, Hq, D, dtype=cache.torch_dtype, device="cuda:0")
    worst, n_points = 0.0, 0
    for t in range(T):
        k, v = gen.step_kv(t)
        if t in check_steps or t >= W:
            q = gen.step_q(t)
            cache.decode_step(-1, q, k, v, out)
        else:
            cache.append_evict(-1, k, v)          # fill: nothing is evicted yet, so there is nothing to encode
        io.step(None)
        if t in check_steps:
            out_h = np64(out[layers][:, seqs])
            for li, l in enumerate(layers):
                for si, b in enumerate(seqs):
                    ref = _oracle_out(gen, l, b, t, io.live(si))
                    worst = max(worst, np.abs(out_h[li, si] - ref).max())
                    n_points += 1
    assert n_points >= 64
    assert worst <= TOL_OUT[c["dtype"]], worst
    # ring state of every layer and sequence, and the state at the samples
    count_want = min(T, W)
    for l in range(L):
        head, count, n_app = cache.get_ring(l)
        assert (count == count_want).all() and (n_app == T).all()
        assert (head == (T - count_want) % W).all()
    for si, b in enumerate(seqs):
        oh, oc, on = io.o.ring(0)
        assert oc[si] == count_want and oh[si] == (T - count_want) % W and on[si] == T
    for l in layers[:3]:
        S = np64(cache.get_state(l)[seqs])
        for si, b in enumerate(seqs[:3]):
            ref = _oracle_state(gen, l, b, [[tok] for tok in io.evicted[si]])
            assert np.abs(S[si] - ref).max() <= TOL_STATE
    assert cache.status() == 0
    cache.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["qwen3b", "qwen7b", "llama8b", "stress-w512-b16", "stress-w1024-b64",
                                  "stress-w4096-b256"])
def test_whole_rollout_integer_parity_two_layers(name):
    """Every step of the rollout: slots, eviction order and counts bit-exact for every sequence; outputs sampled."""
    c = _workload(name)
    L = 2
    B, W, Hq, D, T = c["batch"], c["window"], c["n_q_heads"], c["head_dim"], c["steps"]
    torch.cuda.empty_cache()
    gen, cache = _make_cache(c, L)
    lens = gen.lengths(*c["ragged"]).numpy() if "ragged" in c else np.full(B, T)
    rng = np.random.default_rng(99)
    seqs = sorted({0, B - 1, int(np.argmin(lens)), int(np.argmax(lens)), *rng.integers(0, B, 2).tolist()})
    io = _IntOracle(seqs, W, 1)
    check_steps = {0, W - 1, W, W + 1, 2 * W - 1, 2 * W, T - 1, int(lens.min()) - 1, int(lens.min())}
    check_steps |= {j * W + d for j in range(2, T // W, max(1, T // W // 4)) for d in (-1, 0)}
    check_steps |= {int(lens[b]) - 1 for b in seqs}                  # the last step of each sampled sequence
    check_steps |= set(rng.integers(0, T, 40).tolist())              # >= 256 random (layer, sequence, step) points
    slot = torch.full((T, B), -9, dtype=torch.int32, device="cuda:0")
    first = torch.full((T, B), -9, dtype=torch.int64, device="cuda:0")
    nev = torch.full((T, B), -9, dtype=torch.int32, device="cuda:0")
    out = torch.zeros(L, B, Hq, D, dtype=cache.torch_dtype, device="cuda:0")
    lens_dev = torch.as_tensor(lens, device="cuda:0")
    worst, n_points = 0.0, 0
    slots_or = np.zeros((T, len(seqs)), np.int64)
    for t in range(T):
        ragged = "ragged" in c
        active = (lens_dev > t).to(torch.uint8) if ragged else None
        active_h = (lens > t) if ragged else None
        k, v = gen.step_kv(t)
        # layer 0 through the three calls (append/evict reports its indices), layer 1 through the fused step
        cache.append_evict(0, k[0], v[0], active, slot[t], first[t], nev[t])
        cache.encode(0)
        sl, ev_t, _ = io.step(active_h)
        slots_or[t] = sl
        if t in check_steps:
            q = gen.step_q(t)
            cache.decode_attn(0, q[0], out[0], active)
            cache.decode_step(1, q[1], k[1], v[1], out[1], active)
            out_h = np64(out[:, seqs])
            for si, b in enumerate(seqs):
                if active_h is not None and not active_h[b]:
                    continue
                for l in range(L):
                    ref = _oracle_out(gen, l, b, t, io.live(si))
                    worst = max(worst, np.abs(out_h[l, si] - ref).max())
                    n_points += 1
        else:
            cache.append_evict(1, k[1], v[1], active)
            cache.encode(1)
    assert worst <= TOL_OUT[c["dtype"]], worst
    assert n_points >= 256
    slot_h, first_h, nev_h = slot.cpu().numpy(), first.cpu().numpy(), nev.cpu().numpy()
    # sampled sequences against the oracle's deque / free list, every step
    for si, b in enumerate(seqs):
        assert np.array_equal(slot_h[:, b], slots_or[:, si])
    # every sequence, every step: with FIFO eviction and FIFO slot reuse the t-th token sits in slot t mod W, and from
    # token W on each arrival evicts exactly the token that arrived W steps earlier (both pinned on the oracle in the
    # CPU tests); inactive steps report -1 / 0
    tt = np.arange(T)[:, None]
    act = tt < lens[None, :]
    assert np.array_equal(slot_h, np.where(act, tt % W, -1))
    assert np.array_equal(nev_h, np.where(act & (tt >= W), 1, 0))
    assert np.array_equal(first_h, np.where(act & (tt >= W), tt - W, -1))
    for l in range(L):
        head, count, n_app = cache.get_ring(l)
        assert np.array_equal(n_app.cpu().numpy(), lens)
        assert np.array_equal(count.cpu().numpy(), np.minimum(lens, W))
        assert np.array_equal(head.cpu().numpy(), (lens - np.minimum(lens, W)) % W)
    for l in range(L):
        S = np64(cache.get_state(l)[seqs[:2]])
        for si, b in enumerate(seqs[:2]):
            ref = _oracle_state(gen, l, b, [[tok] for tok in io.evicted[si]])
            assert len(io.evicted[si]) == max(0, lens[b] - W)
            assert np.abs(S[si] - ref).max() <= TOL_STATE
    assert cache.status() == 0
    cache.close()
    torch.cuda.empty_cache()


def test_paper_policy_at_full_size_pinned_prompt_and_quarter_window_chunks():
    """The policy of the paper's runs (Sec. 3.3 / 4.1) on the 7B-shaped workload at full size: the prompt stays
    pinned, the rest of the window slides, a quarter of the window is evicted at once and folded by the
    tensor-core encoder.  Two eviction bursts; outputs and states at sampled points, ring state everywhere."""
    c = _workload("qwen7b")
    L, B, W, Hq, Hkv, D = c["n_layers"], c["batch"], c["window"], c["n_q_heads"], c["n_kv_heads"], c["head_dim"]
    E = W // 4
    torch.cuda.empty_cache()
    gen, cache = _make_cache(c, L, evict_chunk=E)
    assert cache.info()["tensor_core_encode"]
    n_prompt = gen.lengths(64, 700).numpy()
    p_max = int(n_prompt.max())
    Kp = gen.generic(50, 0, (L, B, p_max, Hkv, D), 1.0)
    Vp = gen.generic(51, 0, (L, B, p_max, Hkv, D), 1.0)
    cache.prefill(-1, Kp, Vp, torch.as_tensor(n_prompt, dtype=torch.int32, device="cuda:0"), p_max)
    rng = np.random.default_rng(5)
    seqs = sorted({int(np.argmin(n_prompt)), int(np.argmax(n_prompt)), *rng.integers(0, B, 3).tolist()})
    layers = sorted({0, L - 1, int(rng.integers(0, L))})
    io = _IntOracle(seqs, W, E)
    io.prefill(n_prompt)
    first_full = W - int(n_prompt.max())            # the sequence with the longest prompt fills first
    T = W - int(n_prompt.min()) + E + 3             # every sequence has evicted at least once, most of them twice
    checks = {0, first_full - 1, first_full, first_full + 1, T - 1} | set(rng.integers(first_full, T, 5).tolist())
    out = torch.zeros(L, B, Hq, D, dtype=cache.torch_dtype, device="cuda:0")
    evicted_chunks = [[] for _ in seqs]
    worst, n_points = 0.0, 0
    for j in range(T):
        q = gen.step_q(j)
        k, v = gen.step_kv(j)
        cache.decode_step(-1, q, k, v, out)
        _, ev_t, _ = io.step(None)
        for si, toks in enumerate(ev_t):
            if toks:
                evicted_chunks[si].append(toks)
        if j in checks:
            out_h = np64(out[layers][:, seqs])
            for li, l in enumerate(layers):
                for si, b in enumerate(seqs):
                    n = int(n_prompt[b])
                    # token index t < n is prompt row t; t >= n is the (t - n)-th decoded token of the stream
                    Kd, Vd = gen.token_kv(l, b, [t - n for t in io.live(si)])
                    Kl = np.concatenate([np64(Kp[l, b, :n]), np64(Kd)])
                    Vl = np.concatenate([np64(Vp[l, b, :n]), np64(Vd)])
                    ref, _ = attention_gqa(np64(gen.token_q(l, b, j)), Kl, Vl)
                    worst = max(worst, np.abs(out_h[li, si] - ref).max())
                    n_points += 1
    assert n_points >= 40 and worst <= TOL_OUT["bf16"], worst
    for l in range(L):
        head, count, n_app = cache.get_ring(l)
        assert np.array_equal(cache.get_pinned(l).cpu().numpy(), n_prompt)
        assert np.array_equal(n_app.cpu().numpy(), n_prompt + T)
        cap = W - n_prompt
        jj = T - 1
        want = np.where(jj < cap, jj + 1, cap - E + 1 + (jj - cap) % E)
        assert np.array_equal(count.cpu().numpy(), want)
    for l in layers[:2]:
        S = np64(cache.get_state(l)[seqs])
        for si, b in enumerate(seqs[:3]):
            n = int(n_prompt[b])
            chunks = [[t - n for t in toks] for toks in evicted_chunks[si]]
            assert chunks and all(len(ch) == E for ch in chunks)
            ref = _oracle_state(gen, l, b, chunks)
            assert np.abs(S[si] - ref).max() <= TOL_STATE
    assert cache.status() == 0
    cache.close()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("G", [16, 48, 64])
@pytest.mark.parametrize("ratio", [0.05, 0.25])
def test_ablation_grid_global_tokens_and_eviction_ratio(G, ratio):
    """The paper's ablations as configurations (Sec. 4.3: number of global tokens 16/48/64; appendix: eviction ratios
    5 % to 25 % of the window): 7B head shapes, window 1024, four layers, three eviction bursts."""
    c = {**_workload("qwen7b"), "window": 1024, "batch": 16, "n_global": G}
    L, B, W = 4, c["batch"], c["window"]
    E = max(1, int(round(ratio * W)))
    torch.cuda.empty_cache()
    gen, cache = _make_cache(c, L, evict_chunk=E)
    seqs = [0, 7, 15]
    io = _IntOracle(seqs, W, E)
    T = W + 2 * E + 2
    out = torch.zeros(L, B, c["n_q_heads"], c["head_dim"], dtype=cache.torch_dtype, device="cuda:0")
    chunks = [[] for _ in seqs]
    worst = 0.0
    for t in range(T):
        k, v = gen.step_kv(t)
        if t >= W - 1:
            q = gen.step_q(t)
            cache.decode_step(-1, q, k, v, out)
        else:
            cache.append_evict(-1, k, v)
        _, ev_t, _ = io.step(None)
        for si, toks in enumerate(ev_t):
            if toks:
                chunks[si].append(toks)
        if t in (W - 1, W, W + E, T - 1):
            out_h = np64(out[:, seqs])
            for l in (0, L - 1):
                for si, b in enumerate(seqs):
                    worst = max(worst, np.abs(out_h[l, si] - _oracle_out(gen, l, b, t, io.live(si))).max())
    assert worst <= TOL_OUT["bf16"], worst
    for l in (0, L - 1):
        S = np64(cache.get_state(l)[seqs])
        assert S.shape == (3, G, 32)
        for si, b in enumerate(seqs):
            assert len(chunks[si]) == 3
            assert np.abs(S[si] - _oracle_state(gen, l, b, chunks[si])).max() <= TOL_STATE
    assert cache.status() == 0
    cache.close()
    torch.cuda.empty_cache()


def test_endurance_65536_steps_under_a_1k_window():
    """A 64K-token generation under a 1K window (the length the paper reports reaching, Sec. 4.3): one layer, every
    step through the fused step; slots bit-exact over all 65536 steps, state and outputs against the oracle at the
    end of 64512 evictions."""
    c = {**_workload("qwen7b"), "window": 1024, "batch": 8}
    W, B, T = 1024, 8, 65536
    torch.cuda.empty_cache()
    gen, cache = _make_cache(c, 1)
    out = torch.zeros(1, B, c["n_q_heads"], c["head_dim"], dtype=cache.torch_dtype, device="cuda:0")
    for t in range(T):
        k, v = gen.step_kv(t)
        q = gen.step_q(t)
        cache.decode_step(-1, q, k, v, out)
    head, count, n_app = cache.get_ring(0)
    assert (n_app == T).all() and (count == W).all() and (head == T % W).all()
    for b in (0, B - 1):
        live = list(range(T - W, T))
        ref = _oracle_out(gen, 0, b, T - 1, live)
        assert np.abs(np64(out[0, b]) - ref).max() <= TOL_OUT["bf16"]
    S = np64(cache.get_state(0)[[0]])
    ref = _oracle_state(gen, 0, 0, [[tok] for tok in range(T - W)])
    assert np.abs(S[0] - ref).max() <= TOL_STATE
    assert cache.status() == 0
    cache.close()
    torch.cuda.empty_cache()
