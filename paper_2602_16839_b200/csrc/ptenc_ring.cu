// Ring-buffer KV cache: append / evict (step a1) and reset.
//
// Sec. 3.2 / 3.3: a cache policy prunes the context at every step; when the cache is full the
// earliest tokens are evicted and handed to the encoder.  Sec. 4.1: a chunk of E tokens leaves at
// once.  FIFO eviction with FIFO slot reuse makes the slot of a sequence's t-th token t mod W; the
// kernel never computes t mod W, it walks head/count so that the state stays valid for any E.
#include "ptenc_internal.h"

namespace {

// One CTA per (layer, sequence).  Rows are moved as 16-byte vectors (D*elt is a multiple of 16).
__global__ void __launch_bounds__(128)
k_append_evict(PtencDev p, int l0, const char* __restrict__ k_new, const char* __restrict__ v_new,
               const uint8_t* __restrict__ active, int32_t* slot_out, long long* evict_first_out,
               int32_t* n_evicted_out) {
  const int li = blockIdx.x / p.B;
  const int b = blockIdx.x - li * p.B;
  const int l = l0 + li;
  const long long lb = (long long)l * p.B + b;
  const long long ob = (long long)li * p.B + b;
  const int tid = threadIdx.x;

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

  int head = p.head[lb];
  int count = p.count[lb];
  const long long n = p.n_app[lb];
  const int W = p.W, Hkv = p.Hkv;
  const int ns = p.n_sink[lb];         // pinned prompt entries in slots [0, ns); the ring runs over slots [ns, W)
  const int cap = W - ns;
  const int E = p.E < cap ? p.E : cap; // a chunk never exceeds the sliding capacity
  const int rb = p.D * p.elt;          // bytes per (token, head) row
  const int vpr = rb >> 4;             // 16-byte vectors per row
  if (ns < 0 || cap < 1 || head < 0 || head >= cap || count < 0 || count > cap) {
    if (tid == 0) atomicOr(p.status, PTENC_ST_BAD_INDEX);
    return;
  }

  int m = 0;
  long long first = -1;
  if (count == cap) {
    m = E;
    first = n - count;
    const int per_tok = Hkv * vpr;
    const int total = m * per_tok;
    for (int idx = tid; idx < total; idx += blockDim.x) {
      const int i = idx / per_tok;
      const int rem = idx - i * per_tok;
      const int h = rem / vpr;
      const int v = rem - h * vpr;
      int slot = head + i;
      if (slot >= cap) slot -= cap;
      slot += ns;
      const size_t src = (((size_t)lb * Hkv + h) * W + slot) * rb + (size_t)v * 16;
      const size_t dst = (((size_t)lb * p.E + i) * Hkv + h) * rb + (size_t)v * 16;
      *reinterpret_cast<uint4*>(p.stageK + dst) = *reinterpret_cast<const uint4*>(p.K + src);
      *reinterpret_cast<uint4*>(p.stageV + dst) = *reinterpret_cast<const uint4*>(p.V + src);
    }
    head += E;
    if (head >= cap) head -= cap;
    count -= E;
  }
  // The slot written below is one of the slots staged above when the ring was full.
  __syncthreads();

  int slot = head + count;
  if (slot >= cap) slot -= cap;
  slot += ns;
  for (int idx = tid; idx < Hkv * vpr; idx += blockDim.x) {
    const int h = idx / vpr;
    const int v = idx - h * vpr;
    const size_t src = ((size_t)ob * Hkv + h) * rb + (size_t)v * 16;
    const size_t dst = (((size_t)lb * Hkv + h) * W + slot) * rb + (size_t)v * 16;
    *reinterpret_cast<uint4*>(p.K + dst) = *reinterpret_cast<const uint4*>(k_new + src);
    *reinterpret_cast<uint4*>(p.V + dst) = *reinterpret_cast<const uint4*>(v_new + src);
  }
  if (tid == 0) {
    p.head[lb] = head;
    p.count[lb] = count + 1;
    p.n_app[lb] = n + 1;
    p.n_staged[lb] = m;
    p.evict_first[lb] = first;
    if (slot_out) slot_out[ob] = slot;
    if (evict_first_out) evict_first_out[ob] = first;
    if (n_evicted_out) n_evicted_out[ob] = m;
  }
}

__global__ void k_reset(PtencDev p, const uint8_t* __restrict__ mask, int clear_status) {
  const int l = blockIdx.x / p.B;
  const int b = blockIdx.x - l * p.B;
  if (clear_status && blockIdx.x == 0 && threadIdx.x == 0) { *p.status = 0; *p.work = 0; }
  if (mask != nullptr && mask[b] == 0) return;
  const long long lb = (long long)l * p.B + b;
  if (threadIdx.x == 0) {
    p.head[lb] = 0;
    p.count[lb] = 0;
    p.n_app[lb] = 0;
    p.n_sink[lb] = 0;
    p.n_staged[lb] = 0;
    p.evict_first[lb] = -1;
    if (p.policy == PTENC_POLICY_SCORE) { p.pending[lb] = 0; p.fq_head[lb] = 0; p.fq_count[lb] = 0; }
  }
  if (p.policy == PTENC_POLICY_SCORE)                      // no slot holds a token any more
    for (int i = threadIdx.x; i < p.wb; i += blockDim.x) p.live_bits[lb * p.wb + i] = 0u;
  const int gr = p.G * p.r;
  for (int i = threadIdx.x; i < gr; i += blockDim.x) p.S[lb * gr + i] = p.S0[(long long)l * gr + i];
}

// Prompt entries of an empty sequence: rows go to slots [0, n), which stay pinned for the rollout.
// One CTA per (layer, sequence).
__global__ void __launch_bounds__(256)
k_prefill(PtencDev p, int l0, const char* __restrict__ K_p, const char* __restrict__ V_p,
          const int32_t* __restrict__ n_prompt, int p_max) {
  const int li = blockIdx.x / p.B;
  const int b = blockIdx.x - li * p.B;
  const long long lb = (long long)(l0 + li) * p.B + b;
  const long long ob = (long long)li * p.B + b;
  int n = n_prompt[b];
  if (n <= 0) return;
  // only an empty sequence can take a prompt, and one slot must remain for the sliding part
  if (n > p_max || n >= p.W || p.n_app[lb] != 0 || p.count[lb] != 0 || p.n_sink[lb] != 0) {
    if (threadIdx.x == 0) atomicOr(p.status, PTENC_ST_BAD_INDEX);
    return;
  }
  const int Hkv = p.Hkv, W = p.W;
  const int rb = p.D * p.elt, vpr = rb >> 4;
  const int per_tok = Hkv * vpr;
  for (long long idx = threadIdx.x; idx < (long long)n * per_tok; idx += blockDim.x) {
    const int i = (int)(idx / per_tok);
    const int rem = (int)(idx - (long long)i * per_tok);
    const int h = rem / vpr, v = rem - h * vpr;
    const size_t src = (((size_t)ob * p_max + i) * Hkv + h) * rb + (size_t)v * 16;
    const size_t dst = (((size_t)lb * Hkv + h) * W + i) * rb + (size_t)v * 16;
    *reinterpret_cast<uint4*>(p.K + dst) = *reinterpret_cast<const uint4*>(K_p + src);
    *reinterpret_cast<uint4*>(p.V + dst) = *reinterpret_cast<const uint4*>(V_p + src);
  }
  if (p.policy == PTENC_POLICY_SCORE) {
    // importance-aware policy: the pinned slots are live like any other; they are never candidates for eviction
    for (int i = threadIdx.x; i < n; i += blockDim.x) { p.slot_tok[lb * W + i] = i; p.score[lb * W + i] = 0.f; }
    for (int w = threadIdx.x; w < p.wb; w += blockDim.x) {
      const int lo = w * 32;
      p.live_bits[lb * p.wb + w] = n >= lo + 32 ? 0xffffffffu : (n > lo ? (1u << (n - lo)) - 1u : 0u);
    }
  }
  __syncthreads();          // every thread has read n_app / count / n_sink above before they change
  if (threadIdx.x == 0) {
    p.n_sink[lb] = n;
    p.head[lb] = 0;
    p.count[lb] = 0;
    p.n_app[lb] = n;
    p.n_staged[lb] = 0;
    p.evict_first[lb] = -1;
  }
}

}  // namespace

cudaError_t ptenc_launch_prefill(ptenc_cache* c, int l0, int nl, const void* K_p, const void* V_p,
                                 const int32_t* n_prompt, int p_max, cudaStream_t st) {
  k_prefill<<<nl * c->cfg.batch, 256, 0, st>>>(c->dev, l0, (const char*)K_p, (const char*)V_p, n_prompt, p_max);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t ptenc_launch_append_evict(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new,
                                      const uint8_t* active, int32_t* slot_out, int64_t* evict_first_out,
                                      int32_t* n_evicted_out, cudaStream_t st) {
  k_append_evict<<<nl * c->cfg.batch, 128, 0, st>>>(c->dev, l0, (const char*)k_new, (const char*)v_new, active,
                                                    slot_out, (long long*)evict_first_out, n_evicted_out);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t ptenc_launch_reset(ptenc_cache* c, const uint8_t* seq_mask, cudaStream_t st) {
  k_reset<<<c->cfg.n_layers * c->cfg.batch, 128, 0, st>>>(c->dev, seq_mask, seq_mask == nullptr ? 1 : 0);
  c->launches++;
  return cudaGetLastError();
}
