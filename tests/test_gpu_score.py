"""GPU parity of the importance-aware eviction policy (PTENC_POLICY_SCORE) against the CPU oracle.

Both sides run the same rollout independently.  Compared at every step: which tokens leave and from which slots
(bit for bit), the slot the arriving token takes, attention outputs and log-sum-exps, the per-slot scores, and at the
end the encoder states and the ring bookkeeping.

Which tokens leave is decided by comparing floating-point scores (fp32 on the GPU, float64 in the oracle).  The
oracle reports, for every eviction, the margin between the highest score that left and the lowest candidate score
that stayed.  Where that margin is above the rounding noise of the fp32 scores the decision is unique and must
agree exactly; a sequence that meets a narrower margin and then disagrees is checked for validity (the GPU's choice
differs from the oracle's only by tokens inside the margin) and dropped from the comparison from there on -- the
tests count these and require them to be rare.
"""
import numpy as np
import pytest
import torch

import paper_2602_16839_b200 as pt
from oracle.ptenc_oracle import OracleCache
from ptenc_inputs import CONFIGS, SynthInputs, make_inputs

from _harness import TOL_LSE, TOL_OUT, TOL_STATE, np64

pytestmark = pytest.mark.gpu

SCORE_RTOL, SCORE_ATOL = 2e-5, 2e-6          # fp32 scores against float64 (sums of up to thousands of weights)


def _near(margin, a, b):
    """True when a margin between two scores is within the fp32 noise of scores of that size."""
    return margin <= 4 * (SCORE_RTOL * max(abs(a), abs(b)) + SCORE_ATOL)


class ScorePair:
    """A CUDA cache and an oracle cache under the score policy, same configuration, encoder and inputs."""

    def __init__(self, *, n_layers, batch, n_q_heads, n_kv_heads, head_dim, window, evict_chunk, recent, seed,
                 n_global=16, rank=16, warps=0):
        self.L, self.B, self.Hq, self.Hkv, self.D = n_layers, batch, n_q_heads, n_kv_heads, head_dim
        self.W, self.E = window, evict_chunk
        shape = dict(n_layers=n_layers, batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim)
        self.gen = SynthInputs(seed=seed, dtype="bf16", n_global=n_global, rank=rank, device="cuda:0", **shape)
        cfg = pt.make_config(window=window, evict_chunk=evict_chunk, n_global=n_global, rank=rank, dtype="bf16",
                             policy=pt.binding.POLICY_SCORE, recent=recent, attn_consumer_warps=warps, **shape)
        self.cache = pt.Cache(cfg)
        assert self.cache.info()["tensor_core_attn"]
        self.orc = OracleCache(window=window, evict_chunk=evict_chunk, n_global=n_global, rank=rank, policy="score",
                               recent=recent, **shape)
        for l in range(n_layers):
            P = self.gen.encoder_params(l)
            self.cache.set_encoder(l, P["Wq_a"], P["Wk_a"], P["Wv_a"], P["q_g"], P["k_g"], P["v_g"])
            self.orc.set_encoder(l, **{k: np64(v) for k, v in P.items()})
        self.out = torch.zeros(n_layers, batch, n_q_heads, head_dim, dtype=torch.bfloat16, device="cuda:0")
        self.lse = torch.zeros(n_layers, batch, n_q_heads, dtype=torch.float32, device="cuda:0")
        self.slot = torch.zeros(n_layers, batch, dtype=torch.int32, device="cuda:0")
        self.first = torch.zeros(n_layers, batch, dtype=torch.int64, device="cuda:0")
        self.nev = torch.zeros(n_layers, batch, dtype=torch.int32, device="cuda:0")
        self.diverged = set()                      # (layer, sequence) pairs that met a near tie and took the other side
        self.n_evictions = 0
        self.n_near = 0

    def prefill(self, n_prompt):
        p_max = max(max(n_prompt), 1)
        shape = (self.L, self.B, p_max, self.Hkv, self.D)
        Kp, Vp = self.gen.generic(50, 0, shape, 1.0), self.gen.generic(51, 0, shape, 1.0)
        self.cache.prefill(-1, Kp, Vp, torch.as_tensor(n_prompt, dtype=torch.int32, device="cuda:0"), p_max)
        for l in range(self.L):
            self.orc.prefill(l, np64(Kp[l]), np64(Vp[l]), n_prompt)

    def step(self, t, active=None, fused_layers=()):
        """One decode step on both sides; layers in `fused_layers` go through ptenc_decode_step, the others through
        the three calls (whose append reports slot / first evicted token / count)."""
        q = self.gen.step_q(t)
        k, v = self.gen.step_kv(t)
        act = None if active is None else torch.as_tensor(active, dtype=torch.uint8, device="cuda:0")
        for l in range(self.L):
            if l in fused_layers:
                self.cache.decode_step(l, q[l], k[l], v[l], self.out[l], act)
                self.cache.decode_attn(l, q[l], self.out[l], act, self.lse[l])      # again, for the lse: idempotent
            else:
                self.cache.append_evict(l, k[l], v[l], act, self.slot[l], self.first[l], self.nev[l])
                self.cache.encode(l)
                self.cache.decode_attn(l, q[l], self.out[l], act, self.lse[l])
        qn, kn, vn = np64(q), np64(k), np64(v)
        out_h, lse_h = np64(self.out), np64(self.lse)
        slot_h, first_h, nev_h = self.slot.cpu().numpy(), self.first.cpu().numpy(), self.nev.cpu().numpy()
        for l in range(self.L):
            before = [self.orc.scores(l, b) for b in range(self.B)]
            o_ref, lse_ref, (slots, ev_t, ev_s) = self.orc.decode_step(l, qn[l], kn[l], vn[l], active)
            tok, sl, n = (x.cpu().numpy() for x in self.cache.get_evicted(l))
            for b in range(self.B):
                if (l, b) in self.diverged or (active is not None and not active[b]):
                    continue
                got_t, got_s = tok[b, :n[b]].tolist(), sl[b, :n[b]].tolist()
                if ev_t[b]:
                    self.n_evictions += 1
                if got_t != ev_t[b]:
                    # only tokens inside a rounding-noise margin may differ; then this sequence is on another path
                    assert len(got_t) == len(ev_t[b]), (t, l, b, got_t, ev_t[b])
                    diff = set(got_t) ^ set(ev_t[b])
                    sc = before[b]
                    lo, hi = min(sc[x] for x in diff), max(sc[x] for x in diff)
                    assert _near(hi - lo, lo, hi), (t, l, b, got_t, ev_t[b], lo, hi)
                    self.diverged.add((l, b))
                    self.n_near += 1
                    continue
                assert got_s == ev_s[b], (t, l, b)
                if l not in fused_layers:
                    assert slot_h[l, b] == slots[b] and nev_h[l, b] == len(ev_t[b])
                    assert first_h[l, b] == (ev_t[b][0] if ev_t[b] else -1)
                assert np.abs(out_h[l, b] - o_ref[b]).max() <= TOL_OUT["bf16"], (t, l, b)
                assert np.abs(lse_h[l, b] - lse_ref[b]).max() <= TOL_LSE["bf16"], (t, l, b)

    def check_scores(self):
        """Per-slot scores after the latest append (the mass of the attention that followed it is not folded in on
        either side's stored scores)."""
        for l in range(self.L):
            score, token = (x.cpu().numpy() for x in self.cache.get_scores(l))
            for b in range(self.B):
                if (l, b) in self.diverged:
                    continue
                c = self.orc.seqs[l][b]
                want = {c.slot_of[tok]: (tok, c.score[tok]) for tok in c.live}
                live = {int(s): (int(token[b, s]), float(score[b, s])) for s in np.nonzero(token[b] >= 0)[0]}
                assert set(live) == set(want), (l, b)
                for s, (tok, val) in want.items():
                    assert live[s][0] == tok
                    assert abs(live[s][1] - val) <= SCORE_RTOL * abs(val) + SCORE_ATOL, (l, b, s, live[s][1], val)

    def check_state_and_ring(self):
        for l in range(self.L):
            S = np64(self.cache.get_state(l))
            head, count, n_app = self.cache.get_ring(l)
            oh, oc, on = self.orc.ring(l)
            for b in range(self.B):
                if (l, b) in self.diverged:
                    continue
                assert np.abs(S[b] - self.orc.S[l][b]).max() <= TOL_STATE
                assert int(count[b]) == oc[b] and int(n_app[b]) == on[b]

    def close(self):
        self.cache.close()


@pytest.mark.parametrize("warps", [0, 3])
@pytest.mark.parametrize("W,E,recent,prompts", [(37, 1, 4, None), (96, 24, 16, [0, 33, 64, 95, 80]), (130, 1, 0, None),
                                                (200, 50, 100, [130, 7, 0, 199, 64]), (64, 64, 0, None),
                                                (257, 65, 32, None)])
def test_score_policy_small_shapes(warps, W, E, recent, prompts):
    """Windows with ragged tiles, chunks from one token to the whole window, protected recent windows from none to
    more than the capacity allows, pinned prompts up to W - 1; sequences active at random."""
    p = ScorePair(n_layers=2, batch=5, n_q_heads=14, n_kv_heads=2, head_dim=128, window=W, evict_chunk=E,
                  recent=recent, seed=W + E, warps=warps)
    if prompts is not None:
        p.prefill(prompts)
    rng = np.random.default_rng(W)
    for t in range(2 * W + 3 * E + 20):
        active = None if t % 3 else (rng.random(5) < 0.8).astype(np.uint8)
        p.step(t, active=active, fused_layers=(1,))
        if t % 7 == 0:
            p.check_scores()
    p.check_scores()
    p.check_state_and_ring()
    assert p.n_evictions > 2 * 5 and p.n_near <= 1, (p.n_evictions, p.n_near)
    assert p.cache.status() == 0
    p.close()


def test_score_policy_is_the_sliding_window_when_everything_else_is_protected():
    """recent = W - E protects all but the E oldest tokens: the candidates are exactly what the sliding window
    evicts, so a score-policy cache and a sliding-window cache must agree: slots and states bit for bit, outputs to
    within a few bf16 ulps (the two walk a window's tiles in different orders, so the fp32 sums differ in rounding)."""
    kw = dict(n_layers=2, batch=4, n_q_heads=8, n_kv_heads=2, head_dim=128, window=70, evict_chunk=5, dtype="bf16",
              n_global=16, rank=16)
    gen = SynthInputs(seed=4, device="cuda:0", **{k: v for k, v in kw.items() if k not in ("window", "evict_chunk")})
    a = pt.Cache(pt.make_config(policy=pt.binding.POLICY_SCORE, recent=65, **kw))
    f = pt.Cache(pt.make_config(**kw))
    for l in range(2):
        P = gen.encoder_params(l)
        for c in (a, f):
            c.set_encoder(l, P["Wq_a"], P["Wk_a"], P["Wv_a"], P["q_g"], P["k_g"], P["v_g"])
    oa = torch.zeros(2, 4, 8, 128, dtype=torch.bfloat16, device="cuda:0")
    of = torch.zeros_like(oa)
    sa = torch.zeros(2, 4, dtype=torch.int32, device="cuda:0")
    sf = torch.zeros_like(sa)
    for t in range(200):
        q = gen.step_q(t)
        k, v = gen.step_kv(t)
        if t % 2:
            a.decode_step(-1, q, k, v, oa)
            f.decode_step(-1, q, k, v, of)
        else:
            for c, o, s in ((a, oa, sa), (f, of, sf)):
                c.append_evict(-1, k, v, None, s)
                c.encode(-1)
                c.decode_attn(-1, q, o)
            assert torch.equal(sa, sf)
        assert float((oa.float() - of.float()).abs().max()) <= 4e-3, t
    for l in range(2):
        assert torch.equal(a.get_state(l), f.get_state(l))
    assert a.status() == 0 and f.status() == 0
    a.close(); f.close()


def test_score_policy_keeps_a_token_that_draws_the_attention():
    """Queries aligned with one early token's key: that token collects nearly all the mass of every step and is never
    evicted, while under the sliding window it leaves after W steps."""
    L, B, Hq, Hkv, D, W = 1, 3, 8, 2, 128, 48
    shape = dict(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D)
    gen = SynthInputs(seed=2, dtype="bf16", device="cuda:0", **shape)
    cache = pt.Cache(pt.make_config(window=W, evict_chunk=4, dtype="bf16", policy=pt.binding.POLICY_SCORE, recent=8,
                                    **shape))
    k5, _ = gen.step_kv(5)
    q = k5[:, :, :, None, :].float().expand(L, B, Hkv, Hq // Hkv, D).reshape(L, B, Hq, D).to(torch.bfloat16)
    out = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device="cuda:0")
    for t in range(4 * W):
        k, v = gen.step_kv(t)
        cache.decode_step(-1, q.contiguous(), k, v, out)
    score, token = cache.get_scores(0)
    for b in range(B):
        assert 5 in token[b].tolist()
        s5 = float(score[b][token[b] == 5])
        assert s5 > 0.9 * Hq * (4 * W - 6)
    assert cache.status() == 0
    cache.close()


def test_score_policy_rejects_what_it_does_not_cover():
    bad = [dict(dtype="fp32", head_dim=64), dict(head_dim=32), dict(window=16384), dict(n_q_heads=32, n_kv_heads=2)]
    base = dict(n_layers=1, batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, window=64, dtype="bf16")
    for patch in bad:
        with pytest.raises(pt.PtencError) as e:
            pt.ptenc_workspace_bytes(pt.make_config(policy=pt.binding.POLICY_SCORE, **{**base, **patch}))
        assert e.value.code == pt.binding.PTENC_ESHAPE
    with pytest.raises(pt.PtencError) as e:
        pt.ptenc_workspace_bytes(pt.make_config(recent=3, **base))                  # recent needs the score policy
    assert e.value.code == pt.binding.PTENC_EINVAL
    fifo = pt.Cache(pt.make_config(**base))
    with pytest.raises(pt.PtencError):
        fifo.get_evicted(0)
    fifo.close()


def test_score_policy_full_size_7b_shape():
    """The 7B-shaped workload at full L, B, W under the score policy, through ptenc_decode_step(layer = -1) from the
    first token on (the scores depend on every attention since a token arrived): three sampled (layer, sequence)
    pairs are replayed by the oracle step by step -- evicted tokens and slots bit for bit, outputs, lse, scores,
    states."""
    c = dict(CONFIGS["qwen7b"])
    L, B, W, Hq, Hkv, D = c["n_layers"], c["batch"], c["window"], c["n_q_heads"], c["n_kv_heads"], c["head_dim"]
    recent, steady = 256, 24
    torch.cuda.empty_cache()
    gen = make_inputs(c, seed=0, device="cuda:0")
    cfg = pt.make_config(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W, evict_chunk=1,
                         n_global=c["n_global"], rank=c["rank"], dtype="bf16", policy=pt.binding.POLICY_SCORE,
                         recent=recent)
    cache = pt.Cache(cfg)
    for l in range(L):
        P = gen.encoder_params(l)
        cache.set_encoder(l, P["Wq_a"], P["Wk_a"], P["Wv_a"], P["q_g"], P["k_g"], P["v_g"])
    samples = [(0, 0), (L - 1, B - 1), (13, 77)]
    orcs = []
    for l, b in samples:
        o = OracleCache(n_layers=1, batch=1, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W, evict_chunk=1,
                        n_global=c["n_global"], rank=c["rank"], policy="score", recent=recent)
        o.set_encoder(0, **{k: np64(v) for k, v in gen.encoder_params(l, device="cpu").items()})
        orcs.append(o)
    out = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device="cuda:0")
    lse = torch.zeros(L, B, Hq, dtype=torch.float32, device="cuda:0")
    T = W + steady
    check = {0, 1, W // 2, W - 1, W, W + 1, T - 1}
    alive = [True] * len(samples)
    n_ev = 0
    for t in range(T):
        q = gen.step_q(t)
        k, v = gen.step_kv(t)
        cache.decode_step(-1, q, k, v, out)
        if t in check:
            cache.decode_attn(-1, q, out, None, lse)
        ev = {l: tuple(x.cpu().numpy() for x in cache.get_evicted(l)) for l in {l for l, _ in samples}} if t >= W else {}
        for i, (l, b) in enumerate(samples):
            qq = np64(gen.token_q(l, b, t))[None]
            kk, vv = gen.token_kv(l, b, [t])
            before = orcs[i].scores(0, 0)
            o_ref, lse_ref, (slots, ev_t, ev_s) = orcs[i].decode_step(0, qq, np64(kk), np64(vv))
            if not alive[i]:
                continue
            if t >= W:
                tok, sl, n = ev[l]
                got_t, got_s = tok[b, :n[b]].tolist(), sl[b, :n[b]].tolist()
                n_ev += 1
                if got_t != ev_t[0]:
                    diff = set(got_t) ^ set(ev_t[0])
                    lo, hi = min(before[x] for x in diff), max(before[x] for x in diff)
                    assert _near(hi - lo, lo, hi), (t, l, b, got_t, ev_t[0], lo, hi)
                    alive[i] = False
                    continue
                assert got_s == ev_s[0]
            if t in check:
                assert np.abs(np64(out[l, b]) - o_ref[0]).max() <= TOL_OUT["bf16"]
                assert np.abs(np64(lse[l, b]) - lse_ref[0]).max() <= TOL_LSE["bf16"]
    assert sum(alive) >= 2 and n_ev >= 2 * steady
    for i, (l, b) in enumerate(samples):
        if not alive[i]:
            continue
        score, token = (x.cpu().numpy() for x in cache.get_scores(l))
        cseq = orcs[i].seqs[0][0]
        for tok in cseq.live:
            s = cseq.slot_of[tok]
            assert token[b, s] == tok
            assert abs(score[b, s] - cseq.score[tok]) <= SCORE_RTOL * abs(cseq.score[tok]) + SCORE_ATOL
        assert np.abs(np64(cache.get_state(l)[b]) - orcs[i].S[0][0]).max() <= TOL_STATE
    head, count, n_app = cache.get_ring(0)
    assert (count == W).all() and (n_app == T).all()
    assert cache.status() == 0
    cache.close()
    torch.cuda.empty_cache()
