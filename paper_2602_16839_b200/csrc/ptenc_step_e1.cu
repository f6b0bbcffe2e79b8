// Ring-per-step mode (E = 1): every arriving token evicts exactly one token once the ring is full, so steps a1 and a3
// of a decode step touch one row per sequence.
//
//   k_ring_e1      a1 (Sec. 3.2 / 3.3, sliding-window policy): a warp per (layer, sequence) evicts the oldest token
//                  when the ring is full -- its row goes to the staging area -- writes the arriving token into the
//                  freed slot and advances the ring.  This is all the attention of the same step depends on; it is a
//                  chain of two memory round trips, so the fused decode step runs it alone in front of the attention
//                  kernel and lets the attention kernel's spare warps fold the staged rows (a3) while the K/V stream
//                  runs.
//   k_encode_warp  a3 (Sec. 3.3, Eq. (3)) on its own, for ptenc_encode: a warp per (layer, sequence) folds one row --
//                  the staged one, or a row the caller supplies -- with the routine the attention kernel uses.
#include "ptenc_encode_warp.cuh"
#include "ptenc_internal.h"

namespace {

constexpr int RE_WARPS = 8;                // (layer, sequence) pairs per CTA

__global__ void __launch_bounds__(RE_WARPS * 32)
k_ring_e1(PtencDev p, int l0, int nl, const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
          const uint8_t* __restrict__ active) {
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * RE_WARPS + (threadIdx.x >> 5);
  const bool live = item < nl * p.B;
  const int li = live ? item / p.B : 0, b = live ? item - li * p.B : 0;
  const size_t lb = (size_t)(l0 + li) * p.B + b;
  const size_t ob = (size_t)li * p.B + b;
  const int W = p.W, Hkv = p.Hkv;
  const int vph = p.D >> 3;                          // 16-byte vectors per (token, head) row
  const int vpr = p.d_kv >> 3;                       // and per token (all KV heads)
  // the attention launch behind this kernel may become resident and run its set-up now; it waits for this whole
  // grid before it reads anything
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!live) return;
  // the arriving row does not depend on the ring state: its first two vectors per lane are requested with the ring words
  uint4 nk0 = make_uint4(0u, 0u, 0u, 0u), nv0 = nk0, nk1 = nk0, nv1 = nk0;
  {
    const char* kn = reinterpret_cast<const char*>(k_new) + ob * (size_t)p.d_kv * 2;
    const char* vn = reinterpret_cast<const char*>(v_new) + ob * (size_t)p.d_kv * 2;
    if (lane < vpr) { nk0 = *reinterpret_cast<const uint4*>(kn + (size_t)lane * 16); nv0 = *reinterpret_cast<const uint4*>(vn + (size_t)lane * 16); }
    if (lane + 32 < vpr) { nk1 = *reinterpret_cast<const uint4*>(kn + (size_t)(lane + 32) * 16); nv1 = *reinterpret_cast<const uint4*>(vn + (size_t)(lane + 32) * 16); }
  }

  // every lane reads the ring state itself (same addresses: one request), so nothing waits for a broadcast
  const int act = (active == nullptr) ? 1 : (int)active[b];
  int head = p.head[lb], count = p.count[lb];
  const int ns = p.n_sink[lb];
  const long long n = p.n_app[lb];
  if (act == 0) {
    if (lane == 0) { p.n_staged[lb] = 0; p.evict_first[lb] = -1; }
    return;
  }
  const int cap = W - ns;
  if (ns < 0 || cap < 1 || head < 0 || head >= cap || count < 0 || count > cap) {
    if (lane == 0) atomicOr(p.status, PTENC_ST_BAD_INDEX);
    return;
  }
  int m = 0, ev_slot = 0;
  long long first = -1;
  if (count == cap) {                                // full: the oldest token leaves, its slot is reused at once
    m = 1;
    ev_slot = ns + head;
    first = n - count;
    head = head + 1 == cap ? 0 : head + 1;
    count -= 1;
  }
  int new_slot = head + count;
  if (new_slot >= cap) new_slot -= cap;
  new_slot += ns;
  for (int v = lane; v < vpr; v += 32) {
    const int h = v / vph, vv = v - h * vph;
    const size_t src_new = ((ob * Hkv + h) * p.D) * 2 + (size_t)vv * 16;      // = (ob * d_kv) * 2 + v * 16
    const uint4 nk = v == lane ? nk0 : v == lane + 32 ? nk1
                               : *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(k_new) + src_new);
    const uint4 nv = v == lane ? nv0 : v == lane + 32 ? nv1
                               : *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(v_new) + src_new);
    if (m) {
      // the evicted row is read by the lane that overwrites the same bytes below, so the read comes first
      const size_t src = (((lb * Hkv + h) * W + ev_slot) * p.D) * 2 + (size_t)vv * 16;
      const uint4 k4 = *reinterpret_cast<const uint4*>(p.K + src);
      const uint4 v4 = *reinterpret_cast<const uint4*>(p.V + src);
      const size_t dst = (lb * p.d_kv) * 2 + (size_t)v * 16;            // E = 1: one staged row per sequence
      *reinterpret_cast<uint4*>(p.stageK + dst) = k4;
      *reinterpret_cast<uint4*>(p.stageV + dst) = v4;
    }
    const size_t dst = (((lb * Hkv + h) * W + new_slot) * p.D) * 2 + (size_t)vv * 16;
    *reinterpret_cast<uint4*>(p.K + dst) = nk;
    *reinterpret_cast<uint4*>(p.V + dst) = nv;
  }
  if (lane == 0) {
    p.head[lb] = head;
    p.count[lb] = count + 1;
    p.n_app[lb] = n + 1;
    p.n_staged[lb] = m;
    p.evict_first[lb] = first;
  }
}

__global__ void __launch_bounds__(RE_WARPS * 32)
k_encode_warp(PtencDev p, int l0, int nl, const __nv_bfloat16* __restrict__ Ke, const __nv_bfloat16* __restrict__ Ve,
              const int32_t* __restrict__ n_ev) {
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * RE_WARPS + (threadIdx.x >> 5);
  if (item >= nl * p.B || !p.encode_enabled) return;
  const int li = item / p.B, b = item - li * p.B;
  const int l = l0 + li;
  if (!p.enc_set[l]) return;
  const size_t lb = (size_t)l * p.B + b;
  const size_t ob = (size_t)li * p.B + b;
  const int m = (Ke == nullptr) ? p.n_staged[lb] : n_ev[ob];
  if (m <= 0) return;
  const __nv_bfloat16* rk = (Ke == nullptr) ? reinterpret_cast<const __nv_bfloat16*>(p.stageK) + lb * p.d_kv
                                            : Ke + ob * p.d_kv;
  const __nv_bfloat16* rv = (Ke == nullptr) ? reinterpret_cast<const __nv_bfloat16*>(p.stageV) + lb * p.d_kv
                                            : Ve + ob * p.d_kv;
  encw_fold_row(p, l, lb, rk, rv, lane);
}

}  // namespace

// bf16 storage, one row per sequence, and a state / row size the one-warp routine covers.
bool ptenc_step_e1_usable(const ptenc_cache* c, const void* Ke, int m_max) {
  const PtencDev& p = c->dev;
  if (c->cfg.dtype != PTENC_DTYPE_BF16 || !encw_shape_ok(p.G, p.r, p.d_kv)) return false;
  return Ke == nullptr ? p.E == 1 : m_max == 1;
}

cudaError_t ptenc_launch_ring_e1(ptenc_cache* c, int l0, int nl, const void* k_new, const void* v_new,
                                 const uint8_t* active, cudaStream_t st) {
  const int items = nl * c->cfg.batch;
  k_ring_e1<<<(items + RE_WARPS - 1) / RE_WARPS, RE_WARPS * 32, 0, st>>>(
      c->dev, l0, nl, static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new), active);
  c->launches++;
  return cudaGetLastError();
}

cudaError_t ptenc_launch_encode_e1(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve, const int32_t* n_ev,
                                   cudaStream_t st) {
  const int items = nl * c->cfg.batch;
  k_encode_warp<<<(items + RE_WARPS - 1) / RE_WARPS, RE_WARPS * 32, 0, st>>>(
      c->dev, l0, nl, static_cast<const __nv_bfloat16*>(Ke), static_cast<const __nv_bfloat16*>(Ve), n_ev);
  c->launches++;
  return cudaGetLastError();
}
