// Importance-aware eviction (policy PTENC_POLICY_SCORE): step a1 when the tokens that leave a full cache are the
// ones that received the least attention, not the oldest ones.
//
// Sec. 4.3 (integration with inference-time token dropping) reports that dropping by importance instead of by age
// helps accuracy and leaves the efficient integration into rollouts open.  Here a token's importance is the
// attention mass it has received so far: the softmax weights of Sec. 3.1, summed over all query heads of the layer
// and over the decode steps since the token arrived.  The attention kernel leaves the scaled logits and the
// log-sum-exp of its latest launch in the workspace; the kernel below, run when the next token arrives, turns them
// into weights and adds them to the per-slot scores (once), then -- if the cache is full -- picks the E
// lowest-scoring candidates (unpinned tokens other than the `recent` newest; ties to the older token), stages their
// rows oldest first for the encoder (Sec. 3.3, Eq. (3) is fed exactly as under the sliding window), frees their
// slots in that order, and stores the arriving token in the slot that was freed first.
//
// Slots are no longer a ring: liveness is a bitmap, freed slots sit in a small FIFO, and the attention kernel masks
// its tiles with the bitmap.
#include "ptenc_internal.h"

namespace {

constexpr int SC_THREADS = 256;
constexpr unsigned long long KEY_NONE = ~0ull;

__device__ __forceinline__ float sc_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Ascending bitonic sort of n (a power of two) key/value pairs in shared memory, by the whole CTA.
__device__ void sc_bitonic(unsigned long long* keys, int* vals, int n) {
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      __syncthreads();
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const unsigned long long a = keys[i], b = keys[ixj];
          const bool up = (i & k) == 0;
          if ((a > b) == up) {
            keys[i] = b; keys[ixj] = a;
            const int t = vals[i]; vals[i] = vals[ixj]; vals[ixj] = t;
          }
        }
      }
    }
  }
  __syncthreads();
}

// One CTA per (layer, sequence).  Dynamic shared memory: keys [n2] (8 bytes) and slots [n2] (4 bytes) with n2 the
// window rounded up to a power of two -- used only when more than one token leaves at a time.
__global__ void __launch_bounds__(SC_THREADS)
k_score_step(PtencDev p, int l0, const char* __restrict__ k_new, const char* __restrict__ v_new,
             const uint8_t* __restrict__ active, int32_t* slot_out, long long* evict_first_out,
             int32_t* n_evicted_out, int n2) {
  extern __shared__ __align__(16) unsigned char sc_smem[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(sc_smem);
  int* vals = reinterpret_cast<int*>(keys + n2);
  __shared__ unsigned long long s_best[SC_THREADS / 32];
  __shared__ int s_slot[SC_THREADS / 32];
  __shared__ int s_new_slot;

  const int li = blockIdx.x / p.B;
  const int b = blockIdx.x - li * p.B;
  const int l = l0 + li;
  const size_t lb = (size_t)l * p.B + b;
  const size_t ob = (size_t)li * p.B + b;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int W = p.W, Hkv = p.Hkv, g = p.g;

  if (active != nullptr && active[b] == 0) {
    if (tid == 0) {
      p.n_staged[lb] = 0;
      p.evict_first[lb] = -1;
      if (slot_out) slot_out[ob] = -1;
      if (evict_first_out) evict_first_out[ob] = -1;
      if (n_evicted_out) n_evicted_out[ob] = 0;
    }
    return;
  }

  const int count = p.count[lb];
  const long long n = p.n_app[lb];
  const int ns = p.n_sink[lb];
  const int cap = W - ns;
  if (ns < 0 || cap < 1 || count < 0 || count > cap || n < 0 || n >= 0x7fffffffll || n < (long long)ns + count) {
    if (tid == 0) atomicOr(p.status, PTENC_ST_BAD_INDEX);
    return;
  }
  float* score = p.score + lb * W;
  int* stok = p.slot_tok + lb * W;
  unsigned int* bits = p.live_bits + lb * p.wb;
  const int hi = n < (long long)W ? (int)n : W;            // slots used so far: [0, hi)

  // ---- 1. the latest attention's mass joins the scores (once) ------------------------------------------------------
  if (p.pending[lb] != 0) {
    const float* lse2 = p.lse2 + lb * p.Hq;
    for (int s = ns + tid; s < hi; s += SC_THREADS) {
      if (((bits[s >> 5] >> (s & 31)) & 1u) == 0) continue;
      float acc = 0.f;
      for (int h = 0; h < Hkv; ++h) {
        const float4* src = reinterpret_cast<const float4*>(p.logits + ((lb * Hkv + h) * W + s) * 8);
        const float4 a = src[0], c = src[1];
        const float v[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (i < g) acc += sc_ex2(v[i] - lse2[h * g + i]);
      }
      score[s] += acc;
    }
  }
  __syncthreads();                                         // the scores below are read by other threads
  if (tid == 0) p.pending[lb] = 0;

  // ---- 2. which tokens leave ---------------------------------------------------------------------------------------
  int m = 0;
  if (count == cap) {
    m = p.E < cap ? p.E : cap;
    const int prot = p.recent < cap - m ? p.recent : cap - m;
    const int tok_limit = (int)n - prot;                   // candidates arrived before the `prot` newest tokens
    auto key_of = [&](int s) -> unsigned long long {
      if (s < ns || s >= hi || ((bits[s >> 5] >> (s & 31)) & 1u) == 0) return KEY_NONE;
      const int tok = stok[s];
      if (tok >= tok_limit) return KEY_NONE;
      // scores are sums of non-negative weights, so their bit patterns order like the values; ties go to the
      // smaller token index
      return ((unsigned long long)__float_as_uint(score[s]) << 32) | (unsigned int)tok;
    };
    if (m == 1) {
      unsigned long long best = KEY_NONE;
      int best_slot = -1;
      for (int s = ns + tid; s < hi; s += SC_THREADS) {
        const unsigned long long k = key_of(s);
        if (k < best) { best = k; best_slot = s; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
        const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
        if (ok < best) { best = ok; best_slot = os; }
      }
      if (lane == 0) { s_best[warp] = best; s_slot[warp] = best_slot; }
      __syncthreads();
      if (tid == 0) {
        for (int w = 1; w < SC_THREADS / 32; ++w)
          if (s_best[w] < best) { best = s_best[w]; best_slot = s_slot[w]; }
        vals[0] = best_slot;
        keys[0] = best;
      }
      __syncthreads();
      if (keys[0] == KEY_NONE) m = 0;                      // cannot happen with a consistent state; checked below
    } else {
      for (int s = tid; s < n2; s += SC_THREADS) { keys[s] = s < W ? key_of(s) : KEY_NONE; vals[s] = s; }
      sc_bitonic(keys, vals, n2);                          // the m lowest (score, token) pairs come first
      const bool enough = keys[m - 1] != KEY_NONE;
      __syncthreads();
      if (enough) {
        int m2 = 1;
        while (m2 < m) m2 <<= 1;
        for (int i = tid; i < m2; i += SC_THREADS)         // they leave oldest first: order the chosen by token
          keys[i] = i < m ? (keys[i] & 0xffffffffull) : KEY_NONE;
        sc_bitonic(keys, vals, m2);
      } else {
        m = 0;
      }
    }
    if (m == 0) {                                          // a full cache with no candidate: inconsistent state
      if (tid == 0) atomicOr(p.status, PTENC_ST_BAD_INDEX);
      return;
    }
  }

  // ---- 3. evicted rows -> staging (oldest first), slots freed in that order ------------------------------------------
  const int rb = p.D * p.elt;                              // bytes per (token, head) row
  const int vpr = rb >> 4;
  const int per_tok = Hkv * vpr;
  for (int idx = tid; idx < m * per_tok; idx += SC_THREADS) {
    const int i = idx / per_tok;
    const int rem = idx - i * per_tok;
    const int h = rem / vpr, v = rem - h * vpr;
    const int slot = vals[i];
    const size_t src = ((lb * Hkv + h) * W + slot) * rb + (size_t)v * 16;
    const size_t dst = ((lb * p.E + i) * Hkv + h) * rb + (size_t)v * 16;
    *reinterpret_cast<uint4*>(p.stageK + dst) = *reinterpret_cast<const uint4*>(p.K + src);
    *reinterpret_cast<uint4*>(p.stageV + dst) = *reinterpret_cast<const uint4*>(p.V + src);
  }
  for (int i = tid; i < m; i += SC_THREADS) {
    const int slot = vals[i];
    p.ev_tok[lb * p.E + i] = stok[slot];
    p.ev_slot[lb * p.E + i] = slot;
    p.fq[lb * p.E + i] = slot;
    atomicAnd(&bits[slot >> 5], ~(1u << (slot & 31)));
  }
  __syncthreads();                                         // the slot written below may be one that was just read

  // ---- 4. the arriving token ---------------------------------------------------------------------------------------
  if (tid == 0) {
    int fh = p.fq_head[lb], fc = p.fq_count[lb];
    if (m > 0) { fh = 0; fc = m; }
    int slot = -1;
    if (n < (long long)W && fc == 0) {
      slot = (int)n;                                       // before the first eviction the slots fill in order
    } else if (fc > 0) {
      slot = p.fq[lb * p.E + fh];
      fh += 1;
      fc -= 1;
    }
    if (slot < ns || slot >= W) {
      atomicOr(p.status, PTENC_ST_BAD_INDEX);
      slot = -1;
    } else {
      p.fq_head[lb] = fh;
      p.fq_count[lb] = fc;
      stok[slot] = (int)n;
      score[slot] = 0.f;
      atomicOr(&bits[slot >> 5], 1u << (slot & 31));
      p.count[lb] = count - m + 1;
      p.n_app[lb] = n + 1;
      p.n_staged[lb] = m;
      p.evict_first[lb] = m > 0 ? p.ev_tok[lb * p.E] : -1;
      if (slot_out) slot_out[ob] = slot;
      if (evict_first_out) evict_first_out[ob] = m > 0 ? p.ev_tok[lb * p.E] : -1;
      if (n_evicted_out) n_evicted_out[ob] = m;
    }
    s_new_slot = slot;
  }
  __syncthreads();
  const int slot = s_new_slot;
  if (slot < 0) return;
  for (int idx = tid; idx < per_tok; idx += SC_THREADS) {
    const int h = idx / vpr, v = idx - h * vpr;
    const size_t src = (ob * Hkv + h) * rb + (size_t)v * 16;
    const size_t dst = ((lb * Hkv + h) * W + slot) * rb + (size_t)v * 16;
    *reinterpret_cast<uint4*>(p.K + dst) = *reinterpret_cast<const uint4*>(k_new + src);
    *reinterpret_cast<uint4*>(p.V + dst) = *reinterpret_cast<const uint4*>(v_new + src);
  }
}

// score_out [B][W], token_out [B][W] (-1 where the slot holds no unpinned token) of one layer.
__global__ void k_export_scores(PtencDev p, int layer, float* __restrict__ score_out, int32_t* __restrict__ token_out) {
  const int b = blockIdx.x;
  const size_t lb = (size_t)layer * p.B + b;
  const int ns = p.n_sink[lb];
  for (int s = threadIdx.x; s < p.W; s += blockDim.x) {
    const bool live = s >= ns && ((p.live_bits[lb * p.wb + (s >> 5)] >> (s & 31)) & 1u) != 0;
    score_out[(size_t)b * p.W + s] = live ? p.score[lb * p.W + s] : 0.f;
    token_out[(size_t)b * p.W + s] = live ? p.slot_tok[lb * p.W + s] : -1;
  }
}

int pow2_at_least(int x) {
  int n = 1;
  while (n < x) n <<= 1;
  return n;
}

}  // namespace

size_t ptenc_score_step_smem(const ptenc_config* cfg) {
  const int n2 = cfg->evict_chunk > 1 ? pow2_at_least(cfg->window) : 1;
  return (size_t)n2 * 12;
}

cudaError_t ptenc_launch_score_step(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new,
                                    const uint8_t* active, int32_t* slot_out, int64_t* evict_first_out,
                                    int32_t* n_evicted_out, cudaStream_t st) {
  const size_t smem = ptenc_score_step_smem(&c->cfg);
  static bool attr_done[PTENC_MAX_DEVICES] = {};
  if (ptenc_first_use(attr_done, c->cfg.device)) {
    cudaError_t e = cudaFuncSetAttribute(k_score_step, cudaFuncAttributeMaxDynamicSharedMemorySize, 8192 * 12);
    if (e != cudaSuccess) return e;
  }
  const int n2 = c->cfg.evict_chunk > 1 ? pow2_at_least(c->cfg.window) : 1;
  k_score_step<<<nl * c->cfg.batch, SC_THREADS, smem, st>>>(c->dev, l0, (const char*)k_new, (const char*)v_new, active,
                                                           slot_out, (long long*)evict_first_out, n_evicted_out, n2);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t ptenc_launch_export_scores(ptenc_cache* c, int layer, float* score_out, int32_t* token_out,
                                       cudaStream_t st) {
  k_export_scores<<<c->cfg.batch, 256, 0, st>>>(c->dev, layer, score_out, token_out);
  c->launches++;
  return cudaGetLastError();
}
