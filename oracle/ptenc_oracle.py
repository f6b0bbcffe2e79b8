"""CPU oracle for the Progressive Thought Encoding decode step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 restatement of what the paper defines for one decode step
under a fixed-size cache.  It shares no code with the CUDA path and is imported
only by the tests, by the smoke check and by the benchmark's CPU-baseline leg.

What follows which passage
--------------------------
* cache bookkeeping  : Sec. 3.1 (the cache grows by one entry per decoded token),
  Sec. 3.2 (a cache policy D prunes the context at every step), Sec. 3.3 (decoding
  goes on while the cache has room, then the policy removes the oldest tokens;
  sliding-window policy),
  Sec. 4.1 implementation details (a fraction of the tokens is evicted on
  saturation -> chunk size E).
* attention          : the two unnumbered equations of Sec. 3.1:
  o = softmax(q K^T / sqrt(d)) V over the cache including the new token.
* progressive encode : Eq. (3) of Sec. 3.3 (the bracketed term named S_e), the
  accumulation rule S_e <- Normalize(S_e + S'_e) and the bootstrap initialisation
  from global tokens stated right after it.

Readings taken where the paper is silent or garbled (each is switchable or pinned
in the tests where the mathematics allows):
* the third projection printed in Eq. (3) is W^a_V (the symbol list and the
  initialisation formula use W^a_V);
* q_g is [G, d_q]; W^a_Q is [r, d_q]; W^a_K and W^a_V are [r, d_kv]; a token's
  evicted key/value is the concatenation of all KV heads (d_kv = H_kv * D); the
  state S_e is [G, r] per layer per sequence;
* Normalize: mode 0 divides each of the G rows by max(||row||_2, 1e-12), mode 1
  divides the matrix by max(||S||_F, 1e-12), mode 2 does nothing.
  -- parity unpinned: the paper does not define Normalize.
* concatenated-heads vs per-head encoding -- parity unpinned (paper silent).
* S_0 is not normalised (the initialisation formula carries no Normalize)
  -- parity unpinned.
* no softmax and no scaling inside the encoder (Eq. (3) has neither);
* Delta W = A S_e B with A [d_out, G] and B [r, d_in]; which projection of the model receives it
  is not stated, so the update is applied to a projection given by the caller (d_in, d_out free)
  -- parity unpinned for that choice, the arithmetic itself is pinned;
* order inside a step: evict, append, attend; the live set never exceeds W;
* eviction is FIFO by arrival and freed slots are reused FIFO;
* pinned question tokens (Sec. 3.3, the sliding-window policy keeps the question; Sec. 4.1): a
  prompt of n tokens given to `prefill` occupies the first n of the W cache entries for the whole
  rollout, is attended by every later query, is never evicted and never encoded; the sliding
  window runs over the remaining W - n entries, and a chunk never exceeds that capacity.

* importance-aware eviction (Sec. 4.3, the paragraph on inference-time token dropping: strategies
  that account for token importance are plugged in where the sliding window drops tokens; the
  paper names other systems and defines none of its own).  Reading taken, policy "score": a
  token's importance is the attention mass it has received so far, summed over all query heads
  of the layer (the softmax weights of Sec. 3.1, accumulated step by step; a token starts at
  zero and first receives mass in the step it arrives).  When the cache is full, the tokens that
  leave are the lowest-scoring ones among the candidates -- the unpinned tokens that are not
  among the `recent` newest (the protection shrinks when the capacity leaves no other choice) --
  ties going to the older token; they reach the encoder oldest first and their slots are reused
  in that order.  The mass of the latest attention on a layer is folded into the scores when the
  next token arrives on that layer, so repeating an attention call changes nothing.
  -- parity unpinned for the choice of importance measure; the arithmetic is pinned.

All arithmetic is float64.  Library primitives used as steps: numpy matmul, exp.
"""
from __future__ import annotations

from collections import deque

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------------
# Attention (Sec. 3.1)
# ----------------------------------------------------------------------------------
def attention_one_head(q, K, V):
    """softmax(q K^T / sqrt(d)) V for one query vector.

    q [D]; K, V [n, D].  Returns (o [D], lse) with lse = log sum_j exp(s_j).
    """
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    d = q.shape[0]
    s = (K @ q) / np.sqrt(F64(d))
    smax = np.max(s)
    e = np.exp(s - smax)
    z = np.sum(e)
    p = e / z
    o = p @ V
    return o, smax + np.log(z)


def attention_mass(q, K):
    """Attention mass each cached token receives from one decoded token: the softmax weights of Sec. 3.1 summed over
    all query heads.  q [Hq, D]; K [n, Hkv, D].  Returns [n]; its entries sum to Hq."""
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    Hq, D = q.shape
    g = Hq // K.shape[1]
    mass = np.zeros((K.shape[0],), F64)
    for h in range(Hq):
        s = (K[:, h // g, :] @ q[h]) / np.sqrt(F64(D))
        e = np.exp(s - np.max(s))
        mass += e / np.sum(e)
    return mass


def attention_gqa(q, K, V):
    """Grouped-query decode attention of one token.

    q [Hq, D]; K, V [n, Hkv, D] (the live cache entries, in any order).
    Query head h reads KV head floor(h / (Hq/Hkv)).  Returns (o [Hq, D], lse [Hq]).
    """
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    Hq, D = q.shape
    Hkv = K.shape[1]
    assert Hq % Hkv == 0
    g = Hq // Hkv
    o = np.zeros((Hq, D), F64)
    lse = np.zeros((Hq,), F64)
    for h in range(Hq):
        o[h], lse[h] = attention_one_head(q[h], K[:, h // g, :], V[:, h // g, :])
    return o, lse


# ----------------------------------------------------------------------------------
# Progressive encoder (Sec. 3.3, Eq. (3) and the two sentences after it)
# ----------------------------------------------------------------------------------
def normalize(S, mode=0, eps=1e-12):
    S = np.asarray(S, F64)
    if mode == 0:
        n = np.sqrt(np.sum(S * S, axis=-1, keepdims=True))
        return S / np.maximum(n, eps)
    if mode == 1:
        n = np.sqrt(np.sum(S * S))
        return S / max(n, eps)
    if mode == 2:
        return S.copy()
    raise ValueError("normalize mode")


def latent_queries(Wq_a, q_g):
    """Q_a = W^a_Q q_g for each of the G global queries: [G, r]."""
    return np.asarray(q_g, F64) @ np.asarray(Wq_a, F64).T


def context_state(Qa, Wk_a, Wv_a, K_e, V_e):
    """The bracketed term of Eq. (3): ((W^a_Q q_g)(W^a_K K_e)^T)(W^a_V V_e).

    Qa [G, r]; Wk_a, Wv_a [r, d_kv]; K_e, V_e [m, d_kv] (one row per evicted token).
    Returns [G, r].
    """
    Ka = np.asarray(K_e, F64) @ np.asarray(Wk_a, F64).T      # [m, r]
    Va = np.asarray(V_e, F64) @ np.asarray(Wv_a, F64).T      # [m, r]
    P = np.asarray(Qa, F64) @ Ka.T                           # [G, m]
    return P @ Va                                            # [G, r]


def initial_state(Qa, Wk_a, Wv_a, k_g, v_g):
    """Bootstrap state from the global tokens; zero when there are none (#Global-0)."""
    if k_g is None or v_g is None:
        return np.zeros((Qa.shape[0], np.asarray(Wv_a).shape[0]), F64)
    return context_state(Qa, Wk_a, Wv_a, k_g, v_g)


def encode_update(S, Qa, Wk_a, Wv_a, K_e, V_e, mode=0):
    """S <- Normalize(S + S') with S' the context state of the evicted rows."""
    return normalize(np.asarray(S, F64) + context_state(Qa, Wk_a, Wv_a, K_e, V_e), mode)


# ----------------------------------------------------------------------------------
# Dynamic weight update (Sec. 3.3, Eq. (3) and the sentence after it: theta' = theta + Delta W)
# ----------------------------------------------------------------------------------
def lora_delta(A, S, Bm):
    """Delta W = A S_e B.  A [d_out, G], S [G, r], Bm [r, d_in] -> [d_out, d_in]."""
    return np.asarray(A, F64) @ np.asarray(S, F64) @ np.asarray(Bm, F64)


def lora_apply(y, x, A, S, Bm):
    """Output of a projection whose weight received Delta W, given the output y = W x of the unchanged weight:
    y' = (W + Delta W) x = y + Delta W x, per sequence (each sequence has its own state).
    y [B, d_out], x [B, d_in], S [B, G, r]."""
    y = np.asarray(y, F64).copy()
    x = np.asarray(x, F64)
    for b in range(y.shape[0]):
        y[b] = y[b] + lora_delta(A, S[b], Bm) @ x[b]
    return y


# ----------------------------------------------------------------------------------
# Cache with explicit bookkeeping (no modular index arithmetic anywhere)
# ----------------------------------------------------------------------------------
class _Seq:
    """One (layer, sequence) cache: live tokens in arrival order + FIFO free slots."""

    def __init__(self, W, Hkv, D):
        self.pinned = []                    # token indices of the pinned prompt (never evicted)
        self.live = deque()                 # token indices of the sliding part, oldest first
        self.slot_of = {}                   # token index -> slot
        self.free = deque(range(W))         # free slots, reused in FIFO order
        self.K = np.zeros((W, Hkv, D), F64)
        self.V = np.zeros((W, Hkv, D), F64)
        self.n_appended = 0
        self.score = {}                     # token index -> attention mass received so far (policy "score")
        self.pending = None                 # (token list, mass) of the latest attention, not yet folded in


class OracleCache:
    """Reference decode state for L layers x B sequences."""

    def __init__(self, *, n_layers, batch, n_q_heads, n_kv_heads, head_dim, window,
                 evict_chunk=1, n_global=32, rank=32, normalize_mode=0, encode_enabled=1, policy="fifo", recent=0):
        assert n_q_heads % n_kv_heads == 0 and 1 <= evict_chunk <= window
        assert policy in ("fifo", "score") and recent >= 0
        self.policy, self.recent = policy, recent
        self.L, self.B = n_layers, batch
        self.Hq, self.Hkv, self.D = n_q_heads, n_kv_heads, head_dim
        self.W, self.E = window, evict_chunk
        self.G, self.r = n_global, rank
        self.mode, self.encode_enabled = normalize_mode, encode_enabled
        self.seqs = [[_Seq(window, n_kv_heads, head_dim) for _ in range(batch)] for _ in range(n_layers)]
        self.enc = [None] * n_layers        # (Qa, Wk_a, Wv_a)
        self.S = [None] * n_layers          # [B, G, r]
        self.S0 = [None] * n_layers         # [G, r] initial state of the layer
        self.staged = [[None] * batch for _ in range(n_layers)]   # (K_e, V_e) of the last append
        self.margin = [[np.inf] * batch for _ in range(n_layers)] # policy "score": see _evict_lowest_scores

    # -- set-up ------------------------------------------------------------------------
    def set_encoder(self, layer, Wq_a, Wk_a, Wv_a, q_g, k_g=None, v_g=None):
        Qa = latent_queries(Wq_a, q_g)
        S0 = initial_state(Qa, Wk_a, Wv_a, k_g, v_g)
        self.enc[layer] = (Qa, np.asarray(Wk_a, F64), np.asarray(Wv_a, F64))
        self.S0[layer] = S0
        self.S[layer] = np.repeat(S0[None], self.B, axis=0)

    def reset(self, seq_mask=None):
        """A finished sequence gives its place to a new one: empty cache (no pinned prompt, no tokens) and the
        layer's initial state again, in every layer.  seq_mask None = every sequence."""
        for layer in range(self.L):
            for b in range(self.B):
                if seq_mask is not None and not seq_mask[b]:
                    continue
                self.seqs[layer][b] = _Seq(self.W, self.Hkv, self.D)
                self.staged[layer][b] = None
                if self.S[layer] is not None:
                    self.S[layer][b] = self.S0[layer]

    # -- prompt: pinned entries -----------------------------------------------------------
    def prefill(self, layer, K_p, V_p, n_prompt):
        """The prompt of each sequence enters an empty cache and is pinned: K_p, V_p
        [B, P_max, Hkv, D], n_prompt [B] tokens each (0 = none), at most W - 1."""
        K_p = np.asarray(K_p, F64)
        V_p = np.asarray(V_p, F64)
        for b in range(self.B):
            c = self.seqs[layer][b]
            n = int(n_prompt[b])
            if n == 0:
                continue
            assert c.n_appended == 0 and not c.live and not c.pinned and 0 < n < self.W
            for i in range(n):
                s_new = c.free.popleft()
                c.K[s_new] = K_p[b, i]
                c.V[s_new] = V_p[b, i]
                c.pinned.append(i)
                c.slot_of[i] = s_new
            c.n_appended = n

    # -- a1: append / evict ---------------------------------------------------------------
    def append_evict(self, layer, k_new, v_new, active=None):
        """Token arrives for every active sequence.  Returns per-sequence records:
        slot [B] (-1 inactive), evicted token lists, evicted slot lists."""
        k_new = np.asarray(k_new, F64)
        v_new = np.asarray(v_new, F64)
        slots = np.full((self.B,), -1, np.int64)
        ev_tokens, ev_slots = [], []
        for b in range(self.B):
            c = self.seqs[layer][b]
            self.staged[layer][b] = None
            if active is not None and not active[b]:
                ev_tokens.append([])
                ev_slots.append([])
                continue
            toks, sl = [], []
            capacity = self.W - len(c.pinned)       # entries the sliding part may hold
            if c.pending is not None:               # mass of the latest attention on this layer joins the scores
                for t_tok, m_tok in zip(*c.pending):
                    c.score[t_tok] += m_tok
                c.pending = None
            if len(c.live) == capacity:
                if self.policy == "score":
                    toks, sl = self._evict_lowest_scores(layer, b, capacity)
                else:
                    for _ in range(min(self.E, capacity)):
                        t_old = c.live.popleft()
                        s_old = c.slot_of.pop(t_old)
                        toks.append(t_old)
                        sl.append(s_old)
                        c.free.append(s_old)
                Ke = np.stack([c.K[s].reshape(-1) for s in sl])   # [m, d_kv], age order
                Ve = np.stack([c.V[s].reshape(-1) for s in sl])
                self.staged[layer][b] = (Ke, Ve)
            s_new = c.free.popleft()
            t = c.n_appended
            c.K[s_new] = k_new[b]
            c.V[s_new] = v_new[b]
            c.live.append(t)
            c.slot_of[t] = s_new
            c.n_appended = t + 1
            if self.policy == "score":
                c.score[t] = 0.0
            slots[b] = s_new
            ev_tokens.append(toks)
            ev_slots.append(sl)
        return slots, ev_tokens, ev_slots

    def _evict_lowest_scores(self, layer, b, capacity):
        """Policy "score": of the candidates (unpinned tokens other than the `recent` newest) the m lowest-scoring
        leave, ties to the older token.  Returns (tokens, slots) oldest first and records the margin between the
        highest score that left and the lowest candidate score that stayed."""
        c = self.seqs[layer][b]
        m = min(self.E, capacity)
        protected = min(self.recent, capacity - m)
        candidates = list(c.live)[:capacity - protected]              # arrival order; the newest are protected
        chosen = sorted(candidates, key=lambda tok: (c.score[tok], tok))[:m]
        left = set(chosen)
        stayed = [c.score[tok] for tok in candidates if tok not in left]
        self.margin[layer][b] = (min(stayed) - max(c.score[tok] for tok in chosen)) if stayed else np.inf
        toks, sl = [], []
        for t_old in sorted(chosen):                                  # they leave oldest first
            c.live.remove(t_old)
            s_old = c.slot_of.pop(t_old)
            del c.score[t_old]
            toks.append(t_old)
            sl.append(s_old)
            c.free.append(s_old)
        return toks, sl

    def scores(self, layer, b):
        """{token: attention mass received so far}, the latest attention included, for the unpinned live tokens."""
        c = self.seqs[layer][b]
        out = dict(c.score)
        if c.pending is not None:
            for t_tok, m_tok in zip(*c.pending):
                out[t_tok] += m_tok
        return out

    # -- a3: encode -----------------------------------------------------------------------
    def encode(self, layer, K_e=None, V_e=None):
        """Fold evicted rows into the state.  K_e/V_e: per-sequence list of [m_b, d_kv]
        arrays (or None entries); default = the rows staged by the last append."""
        if not self.encode_enabled:
            return
        if self.enc[layer] is None:        # no encoder set for this layer: nothing to fold into
            return
        Qa, Wk, Wv = self.enc[layer]
        for b in range(self.B):
            if K_e is None:
                st = self.staged[layer][b]
                if st is None:
                    continue
                Ke, Ve = st
            else:
                Ke, Ve = K_e[b], V_e[b]
                if Ke is None or len(Ke) == 0:
                    continue
            self.S[layer][b] = encode_update(self.S[layer][b], Qa, Wk, Wv, Ke, Ve, self.mode)

    # -- a2: attention -----------------------------------------------------------------------
    def decode_attn(self, layer, q, active=None):
        q = np.asarray(q, F64)
        o = np.zeros((self.B, self.Hq, self.D), F64)
        lse = np.zeros((self.B, self.Hq), F64)
        for b in range(self.B):
            if active is not None and not active[b]:
                continue
            c = self.seqs[layer][b]
            if not c.live and not c.pinned:
                continue
            sl = [c.slot_of[t] for t in c.pinned] + [c.slot_of[t] for t in c.live]
            o[b], lse[b] = attention_gqa(q[b], c.K[sl], c.V[sl])
            if self.policy == "score":
                mass = attention_mass(q[b], c.K[sl])
                c.pending = (list(c.live), mass[len(c.pinned):])      # pinned tokens are never candidates
        return o, lse

    # -- a4: one whole step for one layer --------------------------------------------------------
    def decode_step(self, layer, q, k_new, v_new, active=None):
        rec = self.append_evict(layer, k_new, v_new, active)
        self.encode(layer)
        o, lse = self.decode_attn(layer, q, active)
        return o, lse, rec

    # -- views ---------------------------------------------------------------------------------
    def pinned_count(self, layer):
        return np.array([len(self.seqs[layer][b].pinned) for b in range(self.B)], np.int64)

    def ring(self, layer):
        """(oldest sliding token's slot or 0, sliding tokens held, tokens appended incl. the prompt) per sequence."""
        head = np.zeros((self.B,), np.int64)
        count = np.zeros((self.B,), np.int64)
        n_app = np.zeros((self.B,), np.int64)
        for b in range(self.B):
            c = self.seqs[layer][b]
            count[b] = len(c.live)
            n_app[b] = c.n_appended
            head[b] = c.slot_of[c.live[0]] if c.live else 0
        return head, count, n_app
