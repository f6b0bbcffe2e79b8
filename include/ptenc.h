/*
 * ptenc.h -- C ABI of the Progressive Thought Encoding decode hot path (sm_100a).
 *
 * One decode step under a fixed-size KV cache, per layer and per sequence:
 *   a1  ring-buffer append / evict           (Sec. 3.2 cache policy D; Sec. 3.3: decoding fills the
 *                                             cache, then the policy removes the oldest tokens;
 *                                             Sec. 4.1 implementation details: a fraction of the
 *                                             tokens leaves at once when the cache saturates)
 *   a2  grouped-query decode attention       (Sec. 3.1, the two attention equations: the new query
 *                                             attends over the cache including the new token)
 *   a3  progressive encode of evicted tokens (Sec. 3.3, Eq. (3): S' = ((W^a_Q q_g)(W^a_K K_e)^T)(W^a_V V_e);
 *                                             S <- Normalize(S + S'); bootstrap from global tokens)
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 * - Every data pointer is a DEVICE pointer unless the parameter is marked "host".
 *   Tensors are contiguous, row-major in the index order written next to them, 16-byte aligned.
 * - The caller owns all memory.  The library never allocates or frees device memory; its state lives
 *   in the workspace handed to ptenc_cache_create.  The handle itself is a small host object.
 * - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is enqueued on it and
 *   the call returns without synchronising, except where stated.
 * - `layer` is 0..n_layers-1, or -1 meaning "all layers in one call": every tensor argument then gains
 *   a leading [n_layers] dimension.
 * - `active` ([batch] bytes, may be NULL = all active) masks sequences: an inactive sequence's cache and
 *   state are untouched and its output rows are not written.
 * - Return value: PTENC_OK or a negative error code.  Arguments are validated on the host before any
 *   launch; nothing is launched when an error is returned.  Device-side anomalies (a bounded wait that
 *   ran out, an index outside its range) never trap: they set a status word read by ptenc_cache_status.
 * - A handle may be used from one host thread and one stream at a time.  The device the cache was created on
 *   (ptenc_config.device) must be the calling thread's current CUDA device when an entry point is called;
 *   ptenc_cache_create makes it current.
 * - Storage dtype (ptenc_config.dtype) applies to q, k, v, out, the rings and the encoder weights;
 *   the state S, the latent queries Q_a, lse and all accumulation are fp32.
 */
#ifndef PTENC_H
#define PTENC_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define PTENC_API __attribute__((visibility("default")))
#else
#define PTENC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define PTENC_OK              0
#define PTENC_EINVAL         -1   /* NULL pointer, value out of range, layer out of range            */
#define PTENC_ESHAPE         -2   /* shape unsupported (heads not divisible, head_dim, G, r limits)  */
#define PTENC_EALIGN         -3   /* a pointer is not 16-byte aligned (workspace: 1024)              */
#define PTENC_EWORKSPACE     -4   /* workspace smaller than ptenc_workspace_bytes reports            */
#define PTENC_ECUDA          -5   /* a CUDA runtime / driver call failed                             */
#define PTENC_EDEVICE_STATUS -6   /* the device status word is non-zero                              */
#define PTENC_ELIMIT         -7   /* size beyond the built-in scratch of ptenc_attn_rings_static      */

#define PTENC_DTYPE_FP32 0
#define PTENC_DTYPE_BF16 1

#define PTENC_NORM_ROW_L2    0    /* each of the G state rows divided by max(||row||_2, 1e-12)        */
#define PTENC_NORM_FROBENIUS 1    /* whole state divided by max(||S||_F, 1e-12)                       */
#define PTENC_NORM_NONE      2

#define PTENC_POLICY_FIFO    0    /* sliding window: the oldest tokens leave (Sec. 3.3, the policy of the paper's runs) */
#define PTENC_POLICY_SCORE   1    /* the tokens that received the least attention so far leave (Sec. 4.3, token dropping) */

typedef struct ptenc_cache ptenc_cache;   /* opaque host handle */

typedef struct {
  int32_t n_layers;        /* L                                                                    */
  int32_t batch;           /* B  sequences                                                          */
  int32_t n_q_heads;       /* H_q                                                                   */
  int32_t n_kv_heads;      /* H_kv, divides H_q                                                     */
  int32_t head_dim;        /* D, multiple of 8, <= 256                                              */
  int32_t window;          /* W  cache budget: tokens kept per sequence per layer                   */
  int32_t evict_chunk;     /* E  tokens evicted when the cache is full, 1..W                        */
  int32_t n_global;        /* G  number of state vectors (global query tokens), 1..128              */
  int32_t rank;            /* r  length of each state vector, 1..128                                */
  int32_t dtype;           /* PTENC_DTYPE_*                                                         */
  int32_t normalize_mode;  /* PTENC_NORM_*                                                          */
  int32_t encode_enabled;  /* 0: state stays at its initial value ("Global-Only" ablation, Sec. 4.3) */
  int32_t device;          /* CUDA device ordinal the workspace lives on                            */
  int32_t attn_consumer_warps; /* tuning knob of the bf16 tensor-core attention kernel: warps that consume K/V
                                  tiles, 0 = the default (four), 3 or 4 = that many                               */
  int32_t policy;          /* PTENC_POLICY_*: which tokens leave when the cache is full                       */
  int32_t recent;          /* PTENC_POLICY_SCORE only: the newest `recent` tokens are never evicted (0..W-1);
                              must be 0 under PTENC_POLICY_FIFO                                               */
} ptenc_config;

/* Bytes of device workspace a cache with this configuration needs.  Host only, launches nothing.
 * Layout (all inside the workspace): K and V rings [L][B][H_kv][W][D]; ring state head/count (int32)
 * and n_appended (int64) [L][B], pinned-entry counts (int32) [L][B]; evicted-row staging [L][B][E][H_kv*D] for K and for V; state S
 * [L][B][G][r] fp32; per layer Q_a [G][r] fp32 and copies of W^a_K, W^a_V; split-K partials; status.  Under
 * PTENC_POLICY_SCORE also per-slot scores and token indices, a liveness bitmap, the freed-slot queue, and the logits
 * of the latest attention launch [L][B][H_kv][W][8] fp32 (6 % of the rings at head_dim 128). */
PTENC_API int ptenc_workspace_bytes(const ptenc_config* cfg /*host*/, size_t* bytes /*host, out*/);

/* Binds a cache to `dev_workspace` (1024-byte aligned, >= ptenc_workspace_bytes) and zeroes it on
 * `stream`: every ring empty, every state zero, no encoder set.  The workspace must stay allocated
 * until ptenc_cache_destroy.  Copying the workspace is a checkpoint of the whole decode state. */
PTENC_API int ptenc_cache_create(const ptenc_config* cfg /*host*/, void* dev_workspace, size_t bytes,
                       void* stream, ptenc_cache** out /*host, out*/);

/* Frees the host handle only. */
PTENC_API int ptenc_cache_destroy(ptenc_cache* c);

/* Empties the caches of the sequences with seq_mask[b] != 0 (NULL = all) in every layer (ring and pinned prompt
 * entries) and puts their state back to the layer's initial state S_0 (zero when no encoder was set).  With
 * seq_mask == NULL the device status word and the attention kernel's split-unit arrival counters are cleared too,
 * so a cache whose status word reported a launch that gave up (bounded wait ran out, inconsistent ring state)
 * is fully usable again after this call. */
PTENC_API int ptenc_cache_reset(ptenc_cache* c, const uint8_t* seq_mask /*[B], nullable*/, void* stream);

/* Encoder set-up for one layer (Sec. 3.3): stores W^a_K, W^a_V, computes Q_a = q_g W^a_Q^T [G,r] and the
 * initial state S_0 = (Q_a (k_g W^a_K^T)^T)(v_g W^a_V^T) (the bootstrap from global tokens), and sets
 * every sequence's state to S_0 (not normalised).  k_g == NULL or v_g == NULL gives S_0 = 0 (the
 * "#Global-0" ablation).  Shapes: Wq_a [r, H_q*D]; Wk_a, Wv_a [r, H_kv*D]; q_g [G, H_q*D]; k_g, v_g
 * [G, H_kv*D]; all in the storage dtype.  layer = -1 is not accepted here. */
PTENC_API int ptenc_set_encoder(ptenc_cache* c, int layer, const void* Wq_a, const void* Wk_a, const void* Wv_a,
                      const void* q_g, const void* k_g /*nullable*/, const void* v_g /*nullable*/,
                      void* stream);

/* Pinned prompt entries (Sec. 3.3: the sliding-window policy keeps the question tokens; Sec. 4.1).  For every
 * sequence with n_prompt[b] > 0 the first n_prompt[b] rows of K_p, V_p [B, p_max, H_kv, D] (leading [L] when
 * layer == -1) are stored in slots [0, n_prompt[b]) of the sequence's cache and stay there for the whole rollout:
 * every later query attends to them, they are never evicted and never reach the encoder; the ring of
 * ptenc_append_evict then runs over the remaining W - n_prompt[b] slots, and a chunk of evicted tokens never exceeds
 * that capacity.  n_prompt: device int32 [B], the same for every layer.  The sequence must be empty (fresh or reset)
 * and 0 < n_prompt[b] <= min(p_max, W - 1); a sequence that breaks this is left untouched and the device status word
 * gets PTENC_ST_BAD_INDEX (2).  n_prompt[b] == 0 leaves the sequence as it is.  Token indices reported by
 * ptenc_append_evict count the prompt tokens first. */
PTENC_API int ptenc_prefill(ptenc_cache* c, int layer, const void* K_p, const void* V_p,
                            const int32_t* n_prompt /*[B]*/, int32_t p_max, void* stream);

/* Copies one layer's pinned-entry counts to n_pinned [B] (device int32). */
PTENC_API int ptenc_get_pinned(ptenc_cache* c, int layer, int32_t* n_pinned, void* stream);

/* a1.  For each active sequence the token with key/value k_new/v_new [B, H_kv, D] arrives.  If the
 * sequence already holds W tokens, its E oldest tokens are evicted first (FIFO): their K/V rows are
 * copied, oldest first and KV heads concatenated, to the staging area for ptenc_encode, and their slots
 * are freed in that order.  The token is then stored in the oldest free slot.  With FIFO reuse the slot
 * of the t-th token of a sequence is t mod W (with a pinned prompt of n tokens: n + (t - n) mod (W - n), a full
 * cache meaning W - n sliding tokens, and chunks of min(E, W - n)).  Optional outputs ([B] each, nullable): slot_out = slot
 * written (-1 inactive); evict_first_out = index of the oldest evicted token (-1 if none);
 * n_evicted_out = number of tokens evicted (0 or the chunk size). */
PTENC_API int ptenc_append_evict(ptenc_cache* c, int layer, const void* k_new, const void* v_new,
                       const uint8_t* active, int32_t* slot_out, int64_t* evict_first_out,
                       int32_t* n_evicted_out, void* stream);

/* a2.  out[b,h,:] = softmax(q[b,h,:] . K_live^T / sqrt(D)) V_live over the live tokens of KV head
 * floor(h / (H_q/H_kv)), the token appended last included.  q, out [B, H_q, D] (storage dtype);
 * lse_out [B, H_q] fp32 (nullable) = natural-log sum of exp of the scaled scores.  Sequences with an
 * empty cache are skipped like inactive ones. */
PTENC_API int ptenc_decode_attn(ptenc_cache* c, int layer, const void* q, const uint8_t* active,
                      void* out, float* lse_out, void* stream);

/* a3.  Folds evicted tokens into the state: S[b] <- Normalize(S[b] + (Q_a K_a^T) V_a) with
 * K_a = K_e W^a_K^T, V_a = V_e W^a_V^T.  K_e, V_e [B, m_max, H_kv*D] hold n_evicted[b] <= m_max valid rows
 * per sequence; sequences with n_evicted[b] == 0 keep their state.  K_e == NULL (then V_e, n_evicted are
 * ignored): fold the rows staged by the last ptenc_append_evict on this layer; calling it twice folds
 * them twice.  No-op when encode_enabled == 0 or no encoder is set for the layer. */
PTENC_API int ptenc_encode(ptenc_cache* c, int layer, const void* K_e, const void* V_e,
                 const int32_t* n_evicted /*[B]*/, int32_t m_max, void* stream);

/* Dynamic weight update (Sec. 3.3, Eq. (3) and the sentence after it): the state drives a low-rank change of a
 * weight, Delta W = A S_e B, and decoding continues with theta' = theta + Delta W.  Given the output y = W x of the
 * unchanged projection for the token each sequence is decoding, this adds the change for that sequence's current
 * state: y[b,:] += A (S[b] (B x[b,:])); Delta W itself is never formed.  A [d_out, G], Bm [r, d_in], x [B, d_in],
 * y [B, d_out] in/out (leading [L] when layer == -1), all in the storage dtype; accumulation in fp32.  Which
 * projection of the model receives the update is the caller's choice (the paper does not say): d_in and d_out are
 * free, d_in * sizeof(element) must be a multiple of 16 and at most 8192 bytes (PTENC_ESHAPE otherwise).  Rows of inactive sequences are not touched. */
PTENC_API int ptenc_lora_apply(ptenc_cache* c, int layer, const void* A, const void* Bm, const void* x, void* y,
                               const uint8_t* active, int32_t d_in, int32_t d_out, void* stream);

/* a4.  One whole decode step: ptenc_append_evict ; ptenc_encode(staged rows) ; ptenc_decode_attn, with
 * the same results as the three calls.  q, out [B, H_q, D]; k_new, v_new [B, H_kv, D] (leading [L] when
 * layer == -1). */
PTENC_API int ptenc_decode_step(ptenc_cache* c, int layer, const void* q, const void* k_new, const void* v_new,
                      const uint8_t* active, void* out, void* stream);

/* a4 with HOST buffers: the same step as ptenc_decode_step, with q, k_new, v_new, active read from host
 * memory and out written to host memory.  The call enqueues the host-to-device copies into `dev_staging`
 * (device, 256-byte aligned, at least ptenc_host_staging_bytes), the step, and the device-to-host copy of out,
 * and returns without synchronising: synchronise `stream` before reading out_host or reusing the host buffers.
 * To overlap the transfers with the kernels the copies run on two internal copy streams (host objects made on
 * the first call; no device memory); the kernels run on `stream`, and `stream` is made to wait for the last
 * device-to-host copy before the call returns, so a later synchronise of `stream` covers everything.  With
 * layer = -1 the queries and outputs move in groups of layers and each group's attention is its own launch.
 * The staging buffer has two halves which consecutive calls use in turn, so that the uploads of one step can run
 * while the kernels of the step before are still busy.  Consequence for ordering: the host input buffers must hold
 * their values when the call is made (written by the CPU, or by work that has already completed); except for the
 * first call on a staging buffer, the uploads do not wait for earlier work on `stream`.  The staging buffer must
 * not be touched by anything else between calls.  Host buffers should be page-locked for the copies to be
 * asynchronous.  active_host may be NULL. */
PTENC_API int ptenc_host_staging_bytes(ptenc_cache* c, int layer, size_t* bytes /*host, out*/);
PTENC_API int ptenc_decode_step_host(ptenc_cache* c, int layer, const void* q_host, const void* k_new_host,
                                     const void* v_new_host, const uint8_t* active_host, void* out_host,
                                     void* dev_staging, size_t staging_bytes, void* stream);

/* Copies one layer's ring state to device arrays [B] (each nullable): head = slot of the oldest token of the
 * sliding part, counted from the first slot after the pinned entries; count = tokens in the sliding part;
 * n_appended = tokens ever appended (pinned prompt included). */
PTENC_API int ptenc_get_ring(ptenc_cache* c, int layer, int32_t* head, int32_t* count, int64_t* n_appended,
                   void* stream);

/* Copies one layer's state to S_out [B, G, r] fp32 (device). */
PTENC_API int ptenc_get_state(ptenc_cache* c, int layer, float* S_out, void* stream);

/* Importance-aware eviction, PTENC_POLICY_SCORE (Sec. 4.3, integration with inference-time token dropping; the paper
 * plugs in strategies that account for token importance and leaves their efficient integration open -- the measure
 * used here is this library's reading, stated below).
 *
 * A token's score is the attention mass it has received so far: the softmax weights of Sec. 3.1 that every query
 * head of the layer gave it, summed over the heads and over the decode steps since it arrived.  When a token arrives
 * at a full cache, the tokens that leave are the E lowest-scoring candidates -- the unpinned tokens other than the
 * `recent` newest ones (fewer are protected when the capacity leaves no room) -- ties going to the older token.  They
 * are staged for ptenc_encode oldest first, their slots are reused in that order, and everything downstream (a3,
 * a2, the fused step) works as under the sliding window.  Slots are no longer a ring: ptenc_get_ring reports head 0.
 * The mass of the latest attention launch on a layer (ptenc_decode_attn or the attention inside ptenc_decode_step) is
 * folded into the scores when the next token arrives on that layer, so repeating an attention call changes nothing.
 * Shapes: bf16, head_dim 64 or 128, n_q_heads/n_kv_heads <= 8, window <= 8192 (PTENC_ESHAPE otherwise).
 *
 * ptenc_get_evicted: tokens [B][E] (int64, oldest first), slots [B][E], n_evicted [B] of the last append on `layer`;
 * entries past n_evicted[b] are stale.  ptenc_get_scores: score_out [B][W] fp32 and token_out [B][W] (token index
 * held by each slot, -1 for free and pinned slots) as they stand, i.e. without the mass of an attention launch that
 * has not been folded in yet.  Device pointers, each nullable in ptenc_get_evicted.  PTENC_EINVAL under
 * PTENC_POLICY_FIFO. */
PTENC_API int ptenc_get_evicted(ptenc_cache* c, int layer, int64_t* tokens, int32_t* slots, int32_t* n_evicted,
                                void* stream);
PTENC_API int ptenc_get_scores(ptenc_cache* c, int layer, float* score_out, int32_t* token_out, void* stream);

/* Synchronises the device and reads the status word into *dev_status (host).  Returns PTENC_OK when it
 * is zero, PTENC_EDEVICE_STATUS otherwise.  The word is sticky until ptenc_cache_reset(c, NULL, ..). */
PTENC_API int ptenc_cache_status(ptenc_cache* c, int32_t* dev_status /*host, out, nullable*/);

/* Which kernels serve this cache: *tensor_core_attn = 1 for the TMA + tensor-core bf16 attention kernel
 * (bf16, head_dim 64 or 128, H_q/H_kv <= 8), 0 for the shape-generic kernel; *attn_grid = its persistent
 * grid size (0 for the generic kernel); *tensor_core_encode = 1 when chunks of evicted tokens (E >= 2, or
 * ptenc_encode with m_max >= 2) are folded by the tcgen05 kernel (bf16, rank 16/32/64, H_kv*D a multiple of 64),
 * 0 when the shape-generic encoder serves them.  Host only; every output nullable. */
PTENC_API int ptenc_cache_info(ptenc_cache* c, int32_t* tensor_core_attn /*host, out*/,
                               int32_t* attn_grid /*host, out*/, int32_t* tensor_core_encode /*host, out*/);

/* What the next attention launch through this handle would run for `layer` (-1 = all layers in one call), host only,
 * every output nullable: *consumer_warps = warps that consume K/V tiles in the tensor-core kernel (4 unless
 * ptenc_config.attn_consumer_warps says 3), *tile_tokens = tokens per K/V tile, *stages = shared-memory pipeline
 * stages.  All three are 0 when the shape-generic kernel serves the cache. */
PTENC_API int ptenc_attn_launch_info(ptenc_cache* c, int layer, int32_t* consumer_warps /*host, out*/,
                                     int32_t* tile_tokens /*host, out*/, int32_t* stages /*host, out*/);

/* Where one part of the decode state lives inside the workspace (host only): byte offset from the workspace base
 * and size.  The whole workspace is the checkpoint; this map lets a tool save, inspect or patch one part of it.
 * PTENC_EINVAL for an unknown region. */
#define PTENC_REGION_K        0   /* key rings   [L][B][H_kv][W][D], storage dtype                           */
#define PTENC_REGION_V        1   /* value rings                                                             */
#define PTENC_REGION_HEAD     2   /* int32 [L][B]                                                            */
#define PTENC_REGION_COUNT    3   /* int32 [L][B]                                                            */
#define PTENC_REGION_NAPP     4   /* int64 [L][B]                                                            */
#define PTENC_REGION_NPINNED  5   /* int32 [L][B]                                                            */
#define PTENC_REGION_STATE    6   /* fp32  [L][B][G][r]                                                      */
#define PTENC_REGION_TICKETS  7   /* int32 [L][B][H_kv]: split-unit arrival counters of the attention kernel, zero
                                     between launches                                                        */
#define PTENC_REGION_STATUS   8   /* int32: the device status word                                           */
PTENC_API int ptenc_workspace_region(ptenc_cache* c, int region, size_t* offset /*host, out*/,
                                     size_t* bytes /*host, out*/);

/* Timing hook.  The next attention launch made through this handle (by ptenc_decode_attn, ptenc_decode_step
 * or ptenc_decode_step_host) records the two cudaEvent_t (passed as void*) on its stream immediately
 * before and after the attention kernel; the hook is then cleared.  NULL, NULL cancels it. */
PTENC_API int ptenc_time_next_attn(ptenc_cache* c, void* ev_begin, void* ev_end);

/* Launch statistics since creation (host counters): kernels launched by this handle. */
PTENC_API int ptenc_launch_count(ptenc_cache* c, int64_t* n_launches /*host, out*/);

/* Decode attention over KV rings the caller already owns, with no workspace and no allocation of any kind.
 * (The paper has no counterpart: this entry exists for callers, not for the method.)
 *
 * Who it is for: code that cannot obtain device memory at the moment it needs attention -- a serving process
 * that committed all device memory at start-up and froze its allocator, so that a later cudaMalloc can fail or is
 * forbidden; a latency-critical loop that must avoid the device-wide synchronisation cudaMalloc and cudaFree
 * imply.  Such a caller cannot create a ptenc cache (it needs a workspace), so it passes its rings directly.
 * The kernel's scratch (split-K partials, arrival tickets, a status word) lives in a 2,392,320-byte device array
 * that is part of the library image: every GPU that loads the library holds it until the process exits.
 *
 * Computes exactly what ptenc_decode_attn computes with layer = -1, with the same kernel and the same choice of
 * instantiation (consumer warps per launch, see ptenc_attn_launch_info).
 *   cfg      host; n_layers, batch, n_q_heads, n_kv_heads, head_dim, window, dtype, device, attn_consumer_warps are
 *            read.  Only the tensor-core kernel has this variant: dtype bf16, head_dim 64 or 128,
 *            n_q_heads/n_kv_heads <= 8, else PTENC_ESHAPE.  cfg->device must be the calling thread's current device
 *            (PTENC_EINVAL otherwise): the entry does not switch devices.
 *   K, V     device, [L][B][H_kv][W][D] bf16, 16-byte aligned: the rings.  Slots that hold no live token must
 *            contain finite values (e.g. zeros).
 *   head, count  device int32 [L][B]: slot of the oldest live token and number of live tokens of each ring;
 *            live slots are head, head+1, ... (mod W).
 *   q, out   device, [L][B][H_q][D] bf16; active [B] bytes or NULL; lse_out [L][B][H_q] fp32 or NULL.
 *   status_out  device int32 or NULL: receives the kernel's status word (0 = clean) once the call has run.
 *            A ring whose head or count is out of range (head outside [0, W), count outside [0, W]) is skipped:
 *            its output rows are not written and the status word gets bit 2.
 * Limits: n_layers * batch * n_kv_heads <= 65536 units and n_layers * batch * n_kv_heads * window < 2^31 rows, else
 * PTENC_ELIMIT (nothing is launched).
 * The first call on a device resolves the array's device address and sets kernel attributes (once per device,
 * with that device current); make that first call before any stream capture.  Every call on a device shares the
 * one array, and the array keeps the previous call's contents: the entry clears the status word and the tickets on
 * `stream` before the launch, but two calls whose kernels overlap on the GPU (different streams) race on it --
 * serialise them.  Call it from one host thread at a time.  Asynchronous like the other entry points. */
PTENC_API int ptenc_attn_rings_static(const ptenc_config* cfg /*host*/, const void* K, const void* V,
                                      const int32_t* head, const int32_t* count, const void* q,
                                      const uint8_t* active, void* out, float* lse_out, int32_t* status_out,
                                      void* stream);

/* Static string for an error code. */
PTENC_API const char* ptenc_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PTENC_H */
