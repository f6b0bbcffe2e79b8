// Host side of the C ABI declared in include/ptenc.h: validation, workspace carving, launch sequencing.
#include <new>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "ptenc_internal.h"

namespace {

constexpr size_t WS_ALIGN = 1024;
constexpr int PART_SLOTS = 2048;      // split partial slots (two per CTA of the persistent attention grid)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  size_t K, V, head, count, n_app, n_sink, stageK, stageV, n_staged, evict_first, S, S0, Qa, Wk, Wv, enc_set,
      part_acc, part_ml, tickets, status, lora_u, lora_w, total;
  // importance-aware policy only
  size_t slot_tok, score, live_bits, logits, lse2, pending, fq, fq_head, fq_count, ev_tok, ev_slot;
};

int validate_config(const ptenc_config* c) {
  if (c == nullptr) return PTENC_EINVAL;
  if (c->n_layers <= 0 || c->batch <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0 ||
      c->window <= 0)
    return PTENC_EINVAL;
  if (c->evict_chunk < 1 || c->evict_chunk > c->window) return PTENC_EINVAL;
  if (c->dtype != PTENC_DTYPE_FP32 && c->dtype != PTENC_DTYPE_BF16) return PTENC_EINVAL;
  if (c->normalize_mode < 0 || c->normalize_mode > 2) return PTENC_EINVAL;
  if (c->encode_enabled != 0 && c->encode_enabled != 1) return PTENC_EINVAL;
  if (c->device < 0) return PTENC_EINVAL;
  if (c->attn_consumer_warps != 0 && c->attn_consumer_warps != 3 && c->attn_consumer_warps != 4) return PTENC_EINVAL;
  if (c->policy != PTENC_POLICY_FIFO && c->policy != PTENC_POLICY_SCORE) return PTENC_EINVAL;
  if (c->recent < 0 || c->recent >= c->window) return PTENC_EINVAL;
  if (c->policy == PTENC_POLICY_FIFO && c->recent != 0) return PTENC_EINVAL;
  if (c->n_q_heads % c->n_kv_heads != 0) return PTENC_ESHAPE;
  if (c->head_dim % 8 != 0 || c->head_dim > 256) return PTENC_ESHAPE;
  if (c->n_global < 1 || c->n_global > 128 || c->rank < 1 || c->rank > 128) return PTENC_ESHAPE;
  if ((long long)c->n_kv_heads * c->head_dim > 8192) return PTENC_ESHAPE;
  if ((long long)c->window > (1 << 24)) return PTENC_ESHAPE;
  const long long rows = (long long)c->n_layers * c->batch * c->n_kv_heads * c->window;
  if (rows >= (1ll << 31)) return PTENC_ESHAPE;
  if (c->policy == PTENC_POLICY_SCORE) {
    // the attention mass comes out of the tensor-core attention kernel; the selection sorts a window in shared memory
    if (c->dtype != PTENC_DTYPE_BF16 || (c->head_dim != 64 && c->head_dim != 128) ||
        c->n_q_heads / c->n_kv_heads > 8 || c->window > 8192)
      return PTENC_ESHAPE;
  }
  return PTENC_OK;
}

Layout make_layout(const ptenc_config* c) {
  Layout o;
  const size_t elt = c->dtype == PTENC_DTYPE_FP32 ? 4 : 2;
  const size_t L = c->n_layers, B = c->batch, Hkv = c->n_kv_heads, D = c->head_dim, W = c->window;
  const size_t E = c->evict_chunk, G = c->n_global, r = c->rank, d_kv = Hkv * D;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, WS_ALIGN); return at; };
  o.K = take(L * B * Hkv * W * D * elt);
  o.V = take(L * B * Hkv * W * D * elt);
  o.head = take(L * B * 4);
  o.count = take(L * B * 4);
  o.n_app = take(L * B * 8);
  o.n_sink = take(L * B * 4);
  o.stageK = take(L * B * E * d_kv * elt);
  o.stageV = take(L * B * E * d_kv * elt);
  o.n_staged = take(L * B * 4);
  o.evict_first = take(L * B * 8);
  o.S = take(L * B * G * r * 4);
  o.S0 = take(L * G * r * 4);
  o.Qa = take(L * G * r * 4);
  o.Wk = take(L * r * d_kv * elt);
  o.Wv = take(L * r * d_kv * elt);
  o.enc_set = take(L * 4);
  o.part_acc = take((size_t)PART_SLOTS * 8 * D * 4);
  o.part_ml = take((size_t)PART_SLOTS * 16 * 4);
  o.tickets = take(L * B * Hkv * 4);
  o.status = take(64);
  o.lora_u = take((size_t)PTENC_LORA_MAX_PART * L * B * r * 4);     // scratch of the weight update: partial sums of B x
  o.lora_w = take(2 * L * B * G * 2);                               // and S (B x) as two bf16 terms
  o.slot_tok = o.score = o.live_bits = o.logits = o.lse2 = o.pending = o.fq = o.fq_head = o.fq_count = o.ev_tok =
      o.ev_slot = 0;
  if (c->policy == PTENC_POLICY_SCORE) {
    const size_t wb = (W + 63) / 64 * 2, Hq = c->n_q_heads;
    o.slot_tok = take(L * B * W * 4);
    o.score = take(L * B * W * 4);
    o.live_bits = take(L * B * wb * 4);
    o.logits = take(L * B * Hkv * W * 8 * 4);
    o.lse2 = take(L * B * Hq * 4);
    o.pending = take(L * B * 4);
    o.fq = take(L * B * E * 4);
    o.fq_head = take(L * B * 4);
    o.fq_count = take(L * B * 4);
    o.ev_tok = take(L * B * E * 8);
    o.ev_slot = take(L * B * E * 4);
  }
  o.total = off;
  return o;
}

// With PTENC_DEBUG set in the environment, failed CUDA calls are reported on stderr (and every launch is
// followed by a synchronise so the report names the right step).
bool debug_on() {
  static int on = -1;
  if (on < 0) { const char* e = getenv("PTENC_DEBUG"); on = (e != nullptr && e[0] != '\0' && e[0] != '0') ? 1 : 0; }
  return on == 1;
}
bool ok(cudaError_t e, const char* where, cudaStream_t st = nullptr) {
  if (e == cudaSuccess && debug_on()) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess && debug_on()) fprintf(stderr, "[ptenc] %s: %s\n", where, cudaGetErrorString(e));
  return e == cudaSuccess;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

int check_layer(const ptenc_cache* c, int layer, int* l0, int* nl) {
  if (c == nullptr) return PTENC_EINVAL;
  if (layer == -1) { *l0 = 0; *nl = c->cfg.n_layers; return PTENC_OK; }
  if (layer < 0 || layer >= c->cfg.n_layers) return PTENC_EINVAL;
  *l0 = layer; *nl = 1;
  return PTENC_OK;
}

// a1 under whichever eviction policy the cache was created with.
cudaError_t launch_append(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new, const uint8_t* active,
                          int32_t* slot_out, int64_t* evict_first_out, int32_t* n_evicted_out, cudaStream_t st) {
  if (c->cfg.policy == PTENC_POLICY_SCORE)
    return ptenc_launch_score_step(c, l0, nl, k_new, v_new, active, slot_out, evict_first_out, n_evicted_out, st);
  return ptenc_launch_append_evict(c, l0, nl, k_new, v_new, active, slot_out, evict_first_out, n_evicted_out, st);
}

// True when a decode step on this cache runs as "append/evict alone, then the attention kernel with its spare warps
// folding the staged rows": ring-per-step mode on the tensor-core kernels, under either eviction policy (both leave
// the evicted row of a sequence in the same staging slot).
bool step_folds_in_attention(const ptenc_cache* c) {
  return c->cfg.encode_enabled && c->fast_attn && ptenc_step_e1_usable(c, nullptr, 0);
}

// a1 (+ a3 unless the attention launch of the step does it, see above) of a decode step.
bool launch_append_and_encode(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new,
                              const uint8_t* active, cudaStream_t st) {
  if (step_folds_in_attention(c)) {
    if (c->cfg.policy == PTENC_POLICY_SCORE)
      return ok(launch_append(c, l0, nl, k_new, v_new, active, nullptr, nullptr, nullptr, st), "decode_step/append_evict", st);
    return ok(ptenc_launch_ring_e1(c, l0, nl, k_new, v_new, active, st), "decode_step/append_evict", st);
  }
  if (!ok(launch_append(c, l0, nl, k_new, v_new, active, nullptr, nullptr, nullptr, st), "decode_step/append_evict", st))
    return false;
  if (c->cfg.encode_enabled)
    return ok(ptenc_launch_encode(c, l0, nl, nullptr, nullptr, nullptr, 0, st), "decode_step/encode", st);
  return true;
}

cudaError_t launch_attn(ptenc_cache* c, int l0, int nl, const void* q, const uint8_t* active, void* out,
                        float* lse, bool fold_staged, bool early, cudaStream_t st) {
  cudaEvent_t e0 = c->ev_attn_begin, e1 = c->ev_attn_end;
  c->ev_attn_begin = c->ev_attn_end = nullptr;
  if (e0 != nullptr) { cudaEventRecord(e0, st); early = false; }   // an event in between: an ordinary launch
  cudaError_t rc = c->fast_attn ? ptenc_launch_attn_bf16(c, l0, nl, q, active, out, lse, fold_staged, early, st)
                                : ptenc_launch_attn_generic(c, l0, nl, q, active, out, lse, st);
  if (e1 != nullptr) cudaEventRecord(e1, st);
  return rc;
}


// Streams and events of the host-buffer step are made on first use (host objects only, no device memory).
bool ensure_host_pipeline(ptenc_cache* c) {
  if (c->st_in != nullptr) return true;
  bool good = cudaStreamCreateWithFlags(&c->st_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->st_out, cudaStreamNonBlocking) == cudaSuccess;
  auto mk = [&](cudaEvent_t* e) { good = good && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
  mk(&c->ev_start); mk(&c->ev_kv); mk(&c->ev_done); mk(&c->ev_half[0]); mk(&c->ev_half[1]);
  for (int i = 0; i < ptenc_cache::HOST_GROUPS_MAX; ++i) { mk(&c->ev_q[i]); mk(&c->ev_o[i]); }
  return good;
}

void release_host_pipeline(ptenc_cache* c) {
  auto rm = [](cudaEvent_t& e) { if (e != nullptr) { cudaEventDestroy(e); e = nullptr; } };
  rm(c->ev_start); rm(c->ev_kv); rm(c->ev_done); rm(c->ev_half[0]); rm(c->ev_half[1]);
  for (int i = 0; i < ptenc_cache::HOST_GROUPS_MAX; ++i) { rm(c->ev_q[i]); rm(c->ev_o[i]); }
  if (c->st_in != nullptr) { cudaStreamDestroy(c->st_in); c->st_in = nullptr; }
  if (c->st_out != nullptr) { cudaStreamDestroy(c->st_out); c->st_out = nullptr; }
}

}  // namespace

extern "C" {

int ptenc_workspace_bytes(const ptenc_config* cfg, size_t* bytes) {
  if (bytes == nullptr) return PTENC_EINVAL;
  int rc = validate_config(cfg);
  if (rc != PTENC_OK) return rc;
  *bytes = make_layout(cfg).total;
  return PTENC_OK;
}

int ptenc_cache_create(const ptenc_config* cfg, void* ws, size_t bytes, void* stream, ptenc_cache** out) {
  if (out == nullptr) return PTENC_EINVAL;
  *out = nullptr;
  int rc = validate_config(cfg);
  if (rc != PTENC_OK) return rc;
  if (ws == nullptr) return PTENC_EINVAL;
  if ((reinterpret_cast<uintptr_t>(ws) & (WS_ALIGN - 1)) != 0) return PTENC_EALIGN;
  const Layout lay = make_layout(cfg);
  if (bytes < lay.total) return PTENC_EWORKSPACE;

  if (cudaSetDevice(cfg->device) != cudaSuccess) return PTENC_ECUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return PTENC_ECUDA;

  ptenc_cache* c = new (std::nothrow) ptenc_cache();
  if (c == nullptr) return PTENC_EINVAL;
  c->cfg = *cfg;
  c->ws = ws;
  c->ws_bytes = lay.total;
  c->sm_count = prop.multiProcessorCount;
  c->launches = 0;
  c->fast_attn = false;
  c->tc_encode = false;
  c->tc_stage_box = 0;
  c->attn_grid = 0;
  c->ev_attn_begin = c->ev_attn_end = nullptr;
  c->st_in = c->st_out = nullptr;
  c->ev_start = c->ev_kv = c->ev_done = c->ev_half[0] = c->ev_half[1] = nullptr;
  c->host_staging_ptr = nullptr;
  c->host_staging_size = 0;
  c->host_flip = 0;
  for (int i = 0; i < ptenc_cache::HOST_GROUPS_MAX; ++i) c->ev_q[i] = c->ev_o[i] = nullptr;

  PtencDev& d = c->dev;
  char* base = static_cast<char*>(ws);
  d.L = cfg->n_layers; d.B = cfg->batch; d.Hq = cfg->n_q_heads; d.Hkv = cfg->n_kv_heads; d.D = cfg->head_dim;
  d.W = cfg->window; d.E = cfg->evict_chunk; d.G = cfg->n_global; d.r = cfg->rank;
  d.g = d.Hq / d.Hkv; d.d_q = d.Hq * d.D; d.d_kv = d.Hkv * d.D;
  d.dtype = cfg->dtype; d.elt = cfg->dtype == PTENC_DTYPE_FP32 ? 4 : 2;
  d.norm_mode = cfg->normalize_mode; d.encode_enabled = cfg->encode_enabled;
  d.K = base + lay.K; d.V = base + lay.V;
  d.head = reinterpret_cast<int*>(base + lay.head);
  d.count = reinterpret_cast<int*>(base + lay.count);
  d.n_app = reinterpret_cast<long long*>(base + lay.n_app);
  d.n_sink = reinterpret_cast<int*>(base + lay.n_sink);
  d.stageK = base + lay.stageK; d.stageV = base + lay.stageV;
  d.n_staged = reinterpret_cast<int*>(base + lay.n_staged);
  d.evict_first = reinterpret_cast<long long*>(base + lay.evict_first);
  d.S = reinterpret_cast<float*>(base + lay.S);
  d.S0 = reinterpret_cast<float*>(base + lay.S0);
  d.Qa = reinterpret_cast<float*>(base + lay.Qa);
  d.Wk = base + lay.Wk; d.Wv = base + lay.Wv;
  d.enc_set = reinterpret_cast<int*>(base + lay.enc_set);
  d.part_acc = reinterpret_cast<float*>(base + lay.part_acc);
  d.part_ml = reinterpret_cast<float*>(base + lay.part_ml);
  d.tickets = reinterpret_cast<int*>(base + lay.tickets);
  d.part_slots = PART_SLOTS;
  d.status = reinterpret_cast<int*>(base + lay.status);
  d.work = d.status + 4;                               // same 64-byte block as the status word
  c->lora_u = reinterpret_cast<float*>(base + lay.lora_u);
  c->lora_w = reinterpret_cast<__nv_bfloat16*>(base + lay.lora_w);
  d.policy = cfg->policy; d.recent = cfg->recent; d.wb = 0;
  d.slot_tok = nullptr; d.score = nullptr; d.live_bits = nullptr; d.logits = nullptr; d.lse2 = nullptr;
  d.pending = nullptr; d.fq = nullptr; d.fq_head = nullptr; d.fq_count = nullptr; d.ev_tok = nullptr; d.ev_slot = nullptr;
  if (cfg->policy == PTENC_POLICY_SCORE) {
    d.wb = (cfg->window + 63) / 64 * 2;
    d.slot_tok = reinterpret_cast<int*>(base + lay.slot_tok);
    d.score = reinterpret_cast<float*>(base + lay.score);
    d.live_bits = reinterpret_cast<unsigned int*>(base + lay.live_bits);
    d.logits = reinterpret_cast<float*>(base + lay.logits);
    d.lse2 = reinterpret_cast<float*>(base + lay.lse2);
    d.pending = reinterpret_cast<int*>(base + lay.pending);
    d.fq = reinterpret_cast<int*>(base + lay.fq);
    d.fq_head = reinterpret_cast<int*>(base + lay.fq_head);
    d.fq_count = reinterpret_cast<int*>(base + lay.fq_count);
    d.ev_tok = reinterpret_cast<long long*>(base + lay.ev_tok);
    d.ev_slot = reinterpret_cast<int*>(base + lay.ev_slot);
  }

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(ws, 0, lay.total, st) != cudaSuccess) { delete c; return PTENC_ECUDA; }

  cudaError_t e = cudaSuccess;
  c->fast_attn = ptenc_attn_bf16_prepare(c, &e);
  if (!ok(e, "cache_create/attn_prepare")) { delete c; return PTENC_ECUDA; }
  (void)ptenc_encode_tc_prepare(c);
  *out = c;
  return PTENC_OK;
}

int ptenc_cache_destroy(ptenc_cache* c) {
  if (c == nullptr) return PTENC_EINVAL;
  release_host_pipeline(c);
  delete c;
  return PTENC_OK;
}

int ptenc_cache_reset(ptenc_cache* c, const uint8_t* seq_mask, void* stream) {
  if (c == nullptr) return PTENC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (seq_mask == nullptr) {
    // A launch that gave up part-way (a bounded wait ran out, the schedule did not add up) can leave arrival counts
    // of split units behind; the full reset is the documented way back, so it clears them with the status word.
    const PtencDev& d = c->dev;
    if (cudaMemsetAsync(d.tickets, 0, (size_t)d.L * d.B * d.Hkv * 4, st) != cudaSuccess) return PTENC_ECUDA;
  }
  return ptenc_launch_reset(c, seq_mask, st) == cudaSuccess ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_set_encoder(ptenc_cache* c, int layer, const void* Wq_a, const void* Wk_a, const void* Wv_a,
                      const void* q_g, const void* k_g, const void* v_g, void* stream) {
  if (c == nullptr || Wq_a == nullptr || Wk_a == nullptr || Wv_a == nullptr || q_g == nullptr) return PTENC_EINVAL;
  if (layer < 0 || layer >= c->cfg.n_layers) return PTENC_EINVAL;
  if (misaligned(Wq_a) || misaligned(Wk_a) || misaligned(Wv_a) || misaligned(q_g) || misaligned(k_g) ||
      misaligned(v_g))
    return PTENC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const PtencDev& d = c->dev;
  const size_t wbytes = (size_t)d.r * d.d_kv * d.elt;
  if (cudaMemcpyAsync(d.Wk + (size_t)layer * wbytes, Wk_a, wbytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  if (cudaMemcpyAsync(d.Wv + (size_t)layer * wbytes, Wv_a, wbytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  return ptenc_launch_set_encoder(c, layer, Wq_a, q_g, k_g, v_g, st) == cudaSuccess ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_prefill(ptenc_cache* c, int layer, const void* K_p, const void* V_p, const int32_t* n_prompt,
                  int32_t p_max, void* stream) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (K_p == nullptr || V_p == nullptr || n_prompt == nullptr || p_max < 1) return PTENC_EINVAL;
  if (misaligned(K_p) || misaligned(V_p)) return PTENC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return ok(ptenc_launch_prefill(c, l0, nl, K_p, V_p, n_prompt, p_max, st), "prefill", st) ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_get_pinned(ptenc_cache* c, int layer, int32_t* n_pinned, void* stream) {
  if (c == nullptr || layer < 0 || layer >= c->cfg.n_layers || n_pinned == nullptr) return PTENC_EINVAL;
  const size_t B = c->cfg.batch;
  return cudaMemcpyAsync(n_pinned, c->dev.n_sink + layer * B, B * 4, cudaMemcpyDeviceToDevice,
                         static_cast<cudaStream_t>(stream)) == cudaSuccess ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_append_evict(ptenc_cache* c, int layer, const void* k_new, const void* v_new, const uint8_t* active,
                       int32_t* slot_out, int64_t* evict_first_out, int32_t* n_evicted_out, void* stream) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (k_new == nullptr || v_new == nullptr) return PTENC_EINVAL;
  if (misaligned(k_new) || misaligned(v_new)) return PTENC_EALIGN;
  return launch_append(c, l0, nl, k_new, v_new, active, slot_out, evict_first_out, n_evicted_out,
                       static_cast<cudaStream_t>(stream)) == cudaSuccess ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_decode_attn(ptenc_cache* c, int layer, const void* q, const uint8_t* active, void* out, float* lse_out,
                      void* stream) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (q == nullptr || out == nullptr) return PTENC_EINVAL;
  if (misaligned(q) || misaligned(out)) return PTENC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return ok(launch_attn(c, l0, nl, q, active, out, lse_out, false, false, st), "decode_attn", st) ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_encode(ptenc_cache* c, int layer, const void* K_e, const void* V_e, const int32_t* n_evicted,
                 int32_t m_max, void* stream) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (K_e != nullptr) {
    if (V_e == nullptr || n_evicted == nullptr || m_max < 0) return PTENC_EINVAL;
    if (misaligned(K_e) || misaligned(V_e)) return PTENC_EALIGN;
    if (m_max == 0) return PTENC_OK;
  }
  return ptenc_launch_encode(c, l0, nl, K_e, V_e, n_evicted, m_max, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_lora_apply(ptenc_cache* c, int layer, const void* A, const void* Bm, const void* x, void* y,
                     const uint8_t* active, int32_t d_in, int32_t d_out, void* stream) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (A == nullptr || Bm == nullptr || x == nullptr || y == nullptr || d_in < 1 || d_out < 1) return PTENC_EINVAL;
  if (((size_t)d_in * c->dev.elt) % 16 != 0) return PTENC_ESHAPE;     // rows of B and x are read as 16-byte vectors
  if ((size_t)d_in * c->dev.elt > 8 * 1024) return PTENC_ESHAPE;       // eight input rows are staged in shared memory
  if (misaligned(A) || misaligned(Bm) || misaligned(x) || misaligned(y)) return PTENC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return ok(ptenc_launch_lora_apply(c, l0, nl, A, Bm, x, y, active, d_in, d_out, st), "lora_apply", st)
             ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_decode_step(ptenc_cache* c, int layer, const void* q, const void* k_new, const void* v_new,
                      const uint8_t* active, void* out, void* stream) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (q == nullptr || k_new == nullptr || v_new == nullptr || out == nullptr) return PTENC_EINVAL;
  if (misaligned(q) || misaligned(k_new) || misaligned(v_new) || misaligned(out)) return PTENC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!launch_append_and_encode(c, l0, nl, k_new, v_new, active, st)) return PTENC_ECUDA;
  const bool fold = step_folds_in_attention(c);
  if (!ok(launch_attn(c, l0, nl, q, active, out, nullptr, fold, fold && !debug_on(), st), "decode_step/attn", st))
    return PTENC_ECUDA;
  return PTENC_OK;
}

namespace {
struct HostStaging { size_t q, k, v, out, active, total, qbytes, kvbytes; };
HostStaging host_staging(const ptenc_cache* c, int nl) {
  HostStaging h;
  const PtencDev& d = c->dev;
  h.qbytes = (size_t)nl * d.B * d.d_q * d.elt;
  h.kvbytes = (size_t)nl * d.B * d.d_kv * d.elt;
  size_t off = 0;
  auto take = [&](size_t b) { size_t at = off; off = align_up(off + b, 256); return at; };
  h.q = take(h.qbytes); h.k = take(h.kvbytes); h.v = take(h.kvbytes); h.out = take(h.qbytes);
  h.active = take((size_t)d.B);
  h.total = off;
  return h;
}
}  // namespace

int ptenc_host_staging_bytes(ptenc_cache* c, int layer, size_t* bytes) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (bytes == nullptr) return PTENC_EINVAL;
  *bytes = 2 * host_staging(c, nl).total;          // two halves: consecutive steps alternate between them
  return PTENC_OK;
}

int ptenc_decode_step_host(ptenc_cache* c, int layer, const void* q_host, const void* k_new_host,
                           const void* v_new_host, const uint8_t* active_host, void* out_host, void* dev_staging,
                           size_t staging_bytes, void* stream) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  if (q_host == nullptr || k_new_host == nullptr || v_new_host == nullptr || out_host == nullptr ||
      dev_staging == nullptr)
    return PTENC_EINVAL;
  if ((reinterpret_cast<uintptr_t>(dev_staging) & 255) != 0) return PTENC_EALIGN;
  const HostStaging h = host_staging(c, nl);
  const size_t half_bytes = (staging_bytes / 2) & ~(size_t)255;
  if (half_bytes < h.total) return PTENC_EWORKSPACE;
  if (!ensure_host_pipeline(c)) return PTENC_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const PtencDev& d = c->dev;
  auto good = [](cudaError_t e) { return e == cudaSuccess; };

  // Transfers run on two copy streams and join `stream` before the call returns.  Keys/values go first (the append
  // needs them); the queries and the outputs move in groups of layers, each group's attention starting as soon as
  // its queries have landed and its outputs leaving while the next group computes.  Consecutive calls alternate
  // between the two halves of the staging buffer, so the uploads of a step may start while the kernels of the step
  // before are still running: they wait only for their half to be free.  The first call on a staging buffer (or
  // after its size changed) is ordered after everything enqueued on `stream` so far.
  // Layer groups, sized 4, 8, 16, ... from the last layer backwards: the outputs of a group leave while the next,
  // smaller group computes, and only the last four layers' outputs are still to be copied when the kernels end.
  int gb[ptenc_cache::HOST_GROUPS_MAX + 1];
  int ng = 0;
  {
    int ends[ptenc_cache::HOST_GROUPS_MAX + 1];
    int at = nl, size = 4, n = 0;
    ends[n++] = nl;
    while (at > 0 && n < ptenc_cache::HOST_GROUPS_MAX) {
      at = at - size > 0 ? at - size : 0;
      ends[n++] = at;
      size *= 2;
    }
    ends[n - 1] = 0;                                   // the first group takes whatever is left
    ng = n - 1;
    for (int i = 0; i <= ng; ++i) gb[i] = ends[ng - i];
  }
  const bool fresh = c->host_staging_ptr != dev_staging || c->host_staging_size != staging_bytes;
  c->host_staging_ptr = dev_staging;
  c->host_staging_size = staging_bytes;
  const int half = c->host_flip;
  c->host_flip ^= 1;
  char* sb = static_cast<char*>(dev_staging) + (size_t)half * half_bytes;
  if (fresh) {
    if (!good(cudaEventRecord(c->ev_start, st)) || !good(cudaStreamWaitEvent(c->st_in, c->ev_start, 0)) ||
        !good(cudaStreamWaitEvent(c->st_out, c->ev_start, 0)))
      return PTENC_ECUDA;
  } else if (!good(cudaStreamWaitEvent(c->st_in, c->ev_half[half], 0))) {
    return PTENC_ECUDA;
  }
  const uint8_t* act = nullptr;
  if (active_host != nullptr) {
    if (!good(cudaMemcpyAsync(sb + h.active, active_host, c->cfg.batch, cudaMemcpyHostToDevice, c->st_in)))
      return PTENC_ECUDA;
    act = reinterpret_cast<const uint8_t*>(sb + h.active);
  }
  if (!good(cudaMemcpyAsync(sb + h.k, k_new_host, h.kvbytes, cudaMemcpyHostToDevice, c->st_in)) ||
      !good(cudaMemcpyAsync(sb + h.v, v_new_host, h.kvbytes, cudaMemcpyHostToDevice, c->st_in)) ||
      !good(cudaEventRecord(c->ev_kv, c->st_in)))
    return PTENC_ECUDA;
  const size_t q_layer = (size_t)d.B * d.d_q * d.elt;
  for (int g = 0; g < ng; ++g) {
    const int a0 = gb[g], a1 = gb[g + 1];
    if (!good(cudaMemcpyAsync(sb + h.q + a0 * q_layer, static_cast<const char*>(q_host) + a0 * q_layer,
                              (size_t)(a1 - a0) * q_layer, cudaMemcpyHostToDevice, c->st_in)) ||
        !good(cudaEventRecord(c->ev_q[g], c->st_in)))
      return PTENC_ECUDA;
  }
  // a1 + a3 on the caller's stream once the keys/values are on the device
  if (!good(cudaStreamWaitEvent(st, c->ev_kv, 0))) return PTENC_ECUDA;
  if (!launch_append_and_encode(c, l0, nl, sb + h.k, sb + h.v, act, st)) return PTENC_ECUDA;
  // a2 group by group
  for (int g = 0; g < ng; ++g) {
    const int a0 = gb[g], a1 = gb[g + 1];
    if (!good(cudaStreamWaitEvent(st, c->ev_q[g], 0))) return PTENC_ECUDA;
    if (!ok(launch_attn(c, l0 + a0, a1 - a0, sb + h.q + a0 * q_layer, act, sb + h.out + a0 * q_layer, nullptr,
                        step_folds_in_attention(c), false, st),
            "decode_step_host/attn", st))
      return PTENC_ECUDA;
    if (!good(cudaEventRecord(c->ev_o[g], st)) || !good(cudaStreamWaitEvent(c->st_out, c->ev_o[g], 0)) ||
        !good(cudaMemcpyAsync(static_cast<char*>(out_host) + a0 * q_layer, sb + h.out + a0 * q_layer,
                              (size_t)(a1 - a0) * q_layer, cudaMemcpyDeviceToHost, c->st_out)))
      return PTENC_ECUDA;
  }
  if (!good(cudaEventRecord(c->ev_half[half], c->st_out)) || !good(cudaEventRecord(c->ev_done, c->st_out)) ||
      !good(cudaStreamWaitEvent(st, c->ev_done, 0)))
    return PTENC_ECUDA;
  return PTENC_OK;
}

int ptenc_get_ring(ptenc_cache* c, int layer, int32_t* head, int32_t* count, int64_t* n_appended, void* stream) {
  if (c == nullptr || layer < 0 || layer >= c->cfg.n_layers) return PTENC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t B = c->cfg.batch;
  const PtencDev& d = c->dev;
  if (head && cudaMemcpyAsync(head, d.head + layer * B, B * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  if (count && cudaMemcpyAsync(count, d.count + layer * B, B * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  if (n_appended &&
      cudaMemcpyAsync(n_appended, d.n_app + layer * B, B * 8, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  return PTENC_OK;
}

int ptenc_get_state(ptenc_cache* c, int layer, float* S_out, void* stream) {
  if (c == nullptr || layer < 0 || layer >= c->cfg.n_layers || S_out == nullptr) return PTENC_EINVAL;
  const PtencDev& d = c->dev;
  const size_t n = (size_t)d.B * d.G * d.r;
  return cudaMemcpyAsync(S_out, d.S + layer * n, n * 4, cudaMemcpyDeviceToDevice,
                         static_cast<cudaStream_t>(stream)) == cudaSuccess ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_get_evicted(ptenc_cache* c, int layer, int64_t* tokens, int32_t* slots, int32_t* n_evicted, void* stream) {
  if (c == nullptr || layer < 0 || layer >= c->cfg.n_layers) return PTENC_EINVAL;
  if (c->cfg.policy != PTENC_POLICY_SCORE) return PTENC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t B = c->cfg.batch, E = c->cfg.evict_chunk;
  const PtencDev& d = c->dev;
  if (tokens && cudaMemcpyAsync(tokens, d.ev_tok + layer * B * E, B * E * 8, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  if (slots && cudaMemcpyAsync(slots, d.ev_slot + layer * B * E, B * E * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  if (n_evicted &&
      cudaMemcpyAsync(n_evicted, d.n_staged + layer * B, B * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  return PTENC_OK;
}

int ptenc_get_scores(ptenc_cache* c, int layer, float* score_out, int32_t* token_out, void* stream) {
  if (c == nullptr || layer < 0 || layer >= c->cfg.n_layers || score_out == nullptr || token_out == nullptr)
    return PTENC_EINVAL;
  if (c->cfg.policy != PTENC_POLICY_SCORE) return PTENC_EINVAL;
  return ptenc_launch_export_scores(c, layer, score_out, token_out, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? PTENC_OK : PTENC_ECUDA;
}

int ptenc_cache_status(ptenc_cache* c, int32_t* dev_status) {
  if (c == nullptr) return PTENC_EINVAL;
  int32_t st = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return PTENC_ECUDA;
  if (cudaMemcpy(&st, c->dev.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return PTENC_ECUDA;
  if (dev_status) *dev_status = st;
  return st == 0 ? PTENC_OK : PTENC_EDEVICE_STATUS;
}

int ptenc_cache_info(ptenc_cache* c, int32_t* tensor_core_attn, int32_t* attn_grid, int32_t* tensor_core_encode) {
  if (c == nullptr) return PTENC_EINVAL;
  if (tensor_core_attn) *tensor_core_attn = c->fast_attn ? 1 : 0;
  if (attn_grid) *attn_grid = c->fast_attn ? c->attn_grid : 0;
  if (tensor_core_encode) *tensor_core_encode = c->tc_encode ? 1 : 0;
  return PTENC_OK;
}

int ptenc_attn_launch_info(ptenc_cache* c, int layer, int32_t* consumer_warps, int32_t* tile_tokens,
                           int32_t* stages) {
  int l0, nl;
  int rc = check_layer(c, layer, &l0, &nl);
  if (rc != PTENC_OK) return rc;
  int nw = 0, tn = 0, ns = 0;
  if (c->fast_attn) ptenc_attn_bf16_plan(c, nl, &nw, &tn, &ns);
  if (consumer_warps) *consumer_warps = nw;
  if (tile_tokens) *tile_tokens = tn;
  if (stages) *stages = ns;
  return PTENC_OK;
}

int ptenc_workspace_region(ptenc_cache* c, int region, size_t* offset, size_t* bytes) {
  if (c == nullptr || offset == nullptr || bytes == nullptr) return PTENC_EINVAL;
  const Layout lay = make_layout(&c->cfg);
  const size_t elt = c->dev.elt, L = c->dev.L, B = c->dev.B;
  const size_t ring = L * B * (size_t)c->dev.Hkv * c->dev.W * c->dev.D * elt;
  switch (region) {
    case PTENC_REGION_K: *offset = lay.K; *bytes = ring; break;
    case PTENC_REGION_V: *offset = lay.V; *bytes = ring; break;
    case PTENC_REGION_HEAD: *offset = lay.head; *bytes = L * B * 4; break;
    case PTENC_REGION_COUNT: *offset = lay.count; *bytes = L * B * 4; break;
    case PTENC_REGION_NAPP: *offset = lay.n_app; *bytes = L * B * 8; break;
    case PTENC_REGION_NPINNED: *offset = lay.n_sink; *bytes = L * B * 4; break;
    case PTENC_REGION_STATE: *offset = lay.S; *bytes = L * B * (size_t)c->dev.G * c->dev.r * 4; break;
    case PTENC_REGION_TICKETS: *offset = lay.tickets; *bytes = L * B * (size_t)c->dev.Hkv * 4; break;
    case PTENC_REGION_STATUS: *offset = lay.status; *bytes = 4; break;
    default: return PTENC_EINVAL;
  }
  return PTENC_OK;
}

int ptenc_time_next_attn(ptenc_cache* c, void* ev_begin, void* ev_end) {
  if (c == nullptr) return PTENC_EINVAL;
  if ((ev_begin == nullptr) != (ev_end == nullptr)) return PTENC_EINVAL;
  c->ev_attn_begin = static_cast<cudaEvent_t>(ev_begin);
  c->ev_attn_end = static_cast<cudaEvent_t>(ev_end);
  return PTENC_OK;
}

int ptenc_launch_count(ptenc_cache* c, int64_t* n) {
  if (c == nullptr || n == nullptr) return PTENC_EINVAL;
  *n = c->launches;
  return PTENC_OK;
}

const char* ptenc_strerror(int code) {
  switch (code) {
    case PTENC_OK: return "ok";
    case PTENC_EINVAL: return "invalid argument";
    case PTENC_ESHAPE: return "unsupported shape";
    case PTENC_EALIGN: return "misaligned pointer";
    case PTENC_EWORKSPACE: return "workspace too small";
    case PTENC_ECUDA: return "CUDA call failed";
    case PTENC_EDEVICE_STATUS: return "device status word is set";
    case PTENC_ELIMIT: return "size exceeds the built-in scratch limit";
    default: return "unknown error";
  }
}

}  // extern "C"
