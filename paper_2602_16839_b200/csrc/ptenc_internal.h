// Internal declarations shared by the translation units of libptenc (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptenc.h"

// Device status bits (sticky, OR-ed into *status).
#define PTENC_ST_WAIT_TIMEOUT 1   // a bounded mbarrier wait ran out
#define PTENC_ST_BAD_INDEX    2   // an index fell outside its range
#define PTENC_ST_BAD_SCHEDULE 4   // the tile schedule did not add up

// Everything a kernel needs to find the cache's buffers.  Passed by value.
struct PtencDev {
  int L, B, Hq, Hkv, D, W, E, G, r;
  int g, d_q, d_kv;
  int dtype, elt;               // storage dtype and its size in bytes
  int norm_mode, encode_enabled;
  char* K;                      // [L][B][Hkv][W][D]
  char* V;
  int* head;                    // [L][B] slot of the oldest live token
  int* count;                   // [L][B] live tokens
  long long* n_app;             // [L][B] tokens ever appended (pinned prompt included)
  int* n_sink;                  // [L][B] pinned prompt entries: slots [0, n_sink); the ring runs over the rest.
                                //        May be null (= no pinned entries anywhere).
  char* stageK;                 // [L][B][E][d_kv] evicted rows of the last append, oldest first
  char* stageV;
  int* n_staged;                // [L][B] rows staged by the last append (0 or E)
  long long* evict_first;       // [L][B] token index of the oldest staged row (-1 none)
  float* S;                     // [L][B][G][r]
  float* S0;                    // [L][G][r] initial state of the layer
  float* Qa;                    // [L][G][r]
  char* Wk;                     // [L][r][d_kv] storage dtype
  char* Wv;
  int* enc_set;                 // [L]
  float* part_acc;              // [part_slots][8][D] split partial accumulators
  float* part_ml;               // [part_slots][16]  (m2[8], l[8])
  int* tickets;                 // [L][B][Hkv] arrival counters, self-cleaning
  int part_slots;
  int* status;
  int* work;                    // next work item of the running attention launch; zero between launches
  // ---- importance-aware eviction (policy PTENC_POLICY_SCORE); all null / zero under the sliding-window policy -------
  int policy, recent;
  int wb;                       // 32-bit words of one sequence's liveness bitmap
  int* slot_tok;                // [L][B][W] token index held by a slot (meaningful where the slot is live)
  float* score;                 // [L][B][W] attention mass the slot's token has received so far
  unsigned int* live_bits;      // [L][B][wb] bit s set = slot s holds a token (pinned entries included)
  float* logits;                // [L][B][Hkv][W][8] scaled logits (base-2 domain) of the latest attention
  float* lse2;                  // [L][B][Hq] log2-sum-exp2 of the latest attention
  int* pending;                 // [L][B] 1 = the latest attention's mass has not been folded into the scores yet
  int* fq;                      // [L][B][E] freed slots in the order they were freed
  int* fq_head;                 // [L][B] next entry of fq to reuse
  int* fq_count;                // [L][B] entries of fq not reused yet
  long long* ev_tok;            // [L][B][E] tokens evicted by the last append, oldest first
  int* ev_slot;                 // [L][B][E] their slots
};

constexpr int PTENC_LORA_MAX_PART = 16;   // most partial sums of B x per sequence (slices of d_in x parts of a slice)

struct ptenc_cache {
  ptenc_config cfg;
  PtencDev dev;
  size_t ws_bytes;
  void* ws;
  int sm_count;
  int64_t launches;
  bool fast_attn;               // bf16 TMA/tensor-core attention usable for this shape
  CUtensorMap tmK, tmV;         // 2-D maps over the rings: rows = L*B*Hkv*W, cols = D
  int attn_grid;                // persistent grid of the fast attention kernel
  cudaEvent_t ev_attn_begin, ev_attn_end;   // one-shot timing hook around the next attention launch
  // ptenc_decode_step_host: copy streams and events (host objects) that overlap the transfers with the kernels
  static constexpr int HOST_GROUPS_MAX = 8;
  cudaStream_t st_in, st_out;
  cudaEvent_t ev_start, ev_kv, ev_done, ev_q[HOST_GROUPS_MAX], ev_o[HOST_GROUPS_MAX];
  cudaEvent_t ev_half[2];       // a half of the staging buffer is free again (its outputs have left for the host)
  void* host_staging_ptr;       // staging buffer of the last host-buffer step, and its size
  size_t host_staging_size;
  int host_flip;                // half used by the next host-buffer step
  bool tc_encode;               // tensor-core chunk encoder usable for this shape
  CUtensorMap tmWk, tmWv;       // 2-D maps over the encoder weights: rows = L*r, cols = d_kv
  CUtensorMap tmStageK, tmStageV;   // 2-D maps over the staged evicted rows: rows = L*B*E, cols = d_kv
  int tc_stage_box;             // token rows per TMA box of the staged maps
  float* lora_u;                // [PTENC_LORA_MAX_PART][L][B][r] partial sums of B x (scratch of ptenc_lora_apply)
  __nv_bfloat16* lora_w;        // [2][L][B][G] S (B x) split into two bf16 terms (scratch of ptenc_lora_apply)
};

// ---- launchers (each returns a cudaError_t from the launch) -------------------------------------
cudaError_t ptenc_launch_append_evict(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new,
                                      const uint8_t* active, int32_t* slot_out, int64_t* evict_first_out,
                                      int32_t* n_evicted_out, cudaStream_t st);
cudaError_t ptenc_launch_reset(ptenc_cache* c, const uint8_t* seq_mask, cudaStream_t st);
// Importance-aware policy: fold the latest attention's mass into the scores, evict the lowest-scoring candidates
// when the cache is full (rows staged oldest first), store the arriving token in a freed slot.
cudaError_t ptenc_launch_score_step(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new,
                                    const uint8_t* active, int32_t* slot_out, int64_t* evict_first_out,
                                    int32_t* n_evicted_out, cudaStream_t st);
cudaError_t ptenc_launch_export_scores(ptenc_cache* c, int layer, float* score_out, int32_t* token_out,
                                       cudaStream_t st);
size_t ptenc_score_step_smem(const ptenc_config* cfg);
cudaError_t ptenc_launch_prefill(ptenc_cache* c, int l0, int nl, const void* K_p, const void* V_p,
                                 const int32_t* n_prompt, int p_max, cudaStream_t st);
cudaError_t ptenc_launch_encode(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve,
                                const int32_t* n_ev, int m_max, cudaStream_t st);
cudaError_t ptenc_launch_set_encoder(ptenc_cache* c, int layer, const void* Wq, const void* qg,
                                     const void* kg, const void* vg, cudaStream_t st);
cudaError_t ptenc_launch_attn_generic(ptenc_cache* c, int l0, int nl, const void* q, const uint8_t* active,
                                      void* out, float* lse, cudaStream_t st);
// fold_staged: the kernel's spare warps also fold the rows staged by the append of the same step (E = 1) into the
// states of the layers of the call, while the K/V stream runs.
// early: the launch directly follows ptenc_launch_ring_e1 on the same stream and may start while that kernel runs
// (programmatic dependent launch); the attention kernel waits for it before its first read.
cudaError_t ptenc_launch_attn_bf16(ptenc_cache* c, int l0, int nl, const void* q, const uint8_t* active,
                                   void* out, float* lse, bool fold_staged, bool early, cudaStream_t st);
// One evicted token per sequence (E = 1 on the staged path, or caller rows with m_max == 1), bf16, shapes the
// one-warp encoder covers.  ring_e1: the append/evict alone (rows staged); encode_e1: the fold alone.
bool ptenc_step_e1_usable(const ptenc_cache* c, const void* Ke, int m_max);
cudaError_t ptenc_launch_ring_e1(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new,
                                 const uint8_t* active, cudaStream_t st);
cudaError_t ptenc_launch_encode_e1(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve, const int32_t* n_ev,
                                   cudaStream_t st);
// y += A (S (B x)) per sequence with the layer's current states (dynamic weight update, Sec. 3.3).
cudaError_t ptenc_launch_lora_apply(ptenc_cache* c, int l0, int nl, const void* A, const void* Bm, const void* x,
                                    void* y, const uint8_t* active, int d_in, int d_out, cudaStream_t st);
// Chunk encoder on tcgen05 (bf16, rank 16/32/64, d_kv % 64 == 0): tensor maps at create time, launch per call.
bool ptenc_encode_tc_prepare(ptenc_cache* c);
cudaError_t ptenc_launch_encode_tc(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve,
                                   const int32_t* n_ev, int m_max, cudaStream_t st);
// Host-side preparation of the fast attention path (tensor maps, attributes).  Returns false when the
// shape is not covered, in which case the generic kernel serves it.
bool ptenc_attn_bf16_prepare(ptenc_cache* c, cudaError_t* err);
// The instantiation a launch over `nl` layers would use: consumer warps, tokens per tile, pipeline stages.
void ptenc_attn_bf16_plan(const ptenc_cache* c, int nl, int* consumer_warps, int* tile_tokens, int* stages);

// Kernel attributes are per device: a launcher sets them the first time it runs on a device.
constexpr int PTENC_MAX_DEVICES = 64;
inline bool ptenc_first_use(bool (&done)[PTENC_MAX_DEVICES], int device) {
  if (device < 0 || device >= PTENC_MAX_DEVICES) return true;     // unknown ordinal: set the attribute every time
  if (done[device]) return false;
  done[device] = true;
  return true;
}

// ---- small device helpers --------------------------------------------------------------------------
__device__ __forceinline__ float ptenc_to_float(float x) { return x; }
__device__ __forceinline__ float ptenc_to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T ptenc_from_float(float x);
template <> __device__ __forceinline__ float ptenc_from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 ptenc_from_float<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}
