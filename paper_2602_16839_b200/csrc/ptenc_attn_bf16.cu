// Decode attention (step a2), bf16 fast path for sm_100a.
//
// Sec. 3.1: o = softmax(q K^T / sqrt(d)) V over the live cache entries (the new token included), for
// the g = H_q / H_kv query heads that share one KV head.  The path is bound by HBM: every live K/V byte
// is read once per step and there is no reuse between steps.
//
// Design
//  * Persistent grid, one CTA per SM.  The work is the K/V tiles (32 tokens at head_dim 128, 64 at head_dim 64) of
//    every (layer, sequence, KV head) unit that has live tokens, cut into work items: a whole unit, or -- when the
//    call is small -- pieces of a unit, so that every CTA gets several items (split-K sized to the machine).  CTAs
//    take items from a counter in global memory as they go: SMs do not stream at the same rate, and with fixed equal
//    shares the slowest SM set the time of the launch.
//  * A producer warp streams K and V tiles with TMA (cp.async.bulk.tensor, 128-byte swizzle; plain per-CTA loads
//    of this GPU's own memory) into a ring of shared-memory stages guarded by full/empty mbarriers.
//  * Each consumer warp owns whole tiles (tile i of an item goes to warp i mod NW, which cycles through its own
//    STAGES / NW pipeline stages, so a stage always has the same consumer warp and its full/empty barriers advance
//    one phase per visit -- a warp can never be a phase ahead of a barrier it polls).  The two products run on
//    warp-level bf16 mma (m16n8k16, fp32 accumulate) only to keep the FP32 pipes free, in transposed form so that
//    all 16 rows of the mma carry data: S^T = K Q^T (rows = 16 tokens, columns = the g <= 8 query heads) and
//    O^T += V^T P^T (rows = 16 head dims, columns = heads); P^T is turned from accumulator layout into a B
//    fragment with movmatrix.  Online softmax per head, reduced over the lanes' token rows; per-warp (m, l, O).
//  * Per unit the warps' partials are merged in shared memory (fp32).  A unit that is split between CTAs
//    goes through fp32 partials in global scratch; the CTA that arrives last (atomic ticket) combines them.
//    No CTA ever waits for another.
//  * Every mbarrier wait is bounded; when one runs out the CTA raises a status bit, stops waiting and runs
//    to completion on whatever is in shared memory, so barriers stay matched and nothing hangs.
//  * Two more warps per CTA are the step's encoders (Sec. 3.3, Eq. (3)): in a fused ring-per-step decode step it folds
//    the rows that the append of the same step evicted into the states, a (layer, sequence) at a time each, while the
//    other warps stream K/V.  The attention of a step does not read the state, so the two are independent; the
//    encoder's traffic (one evicted row, the encoder weights from L2, 8 KiB of state) is noise beside the K/V stream,
//    and its chain of dependent memory round trips no longer sits in front of the attention.
#include <math.h>
#include <string.h>

#include "ptenc_encode_warp.cuh"
#include "ptenc_internal.h"

// Compile-time tunables of the D = 128 kernel (defaults: 32-token tiles = 16 KiB stages, three per consumer warp).
#ifndef PTENC_ATTN_TILE_N_128
#define PTENC_ATTN_TILE_N_128 32
#endif
#ifndef PTENC_ATTN_STAGES_128
#define PTENC_ATTN_STAGES_128 12
#endif
#ifndef PTENC_ATTN_NW
#define PTENC_ATTN_NW 4
#endif
#ifndef PTENC_ATTN_CTAS_PER_SM
#define PTENC_ATTN_CTAS_PER_SM 1
#endif
#ifndef PTENC_ATTN_ENC_WARPS
#define PTENC_ATTN_ENC_WARPS 2          // warps that fold staged rows while the others stream K/V
#endif
#ifndef PTENC_ATTN_L2PROMO
#define PTENC_ATTN_L2PROMO CU_TENSOR_MAP_L2_PROMOTION_L2_256B
#endif

namespace {

constexpr uint32_t WAIT_POLLS = 4000000;   // bounded wait: tries of up to a microsecond each before giving up

// ------------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait.  try_wait lets the hardware park the thread (up to the hint, in ns) instead of spinning on the
// barrier; the loop bounds the total.  Returns false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < WAIT_POLLS; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    if (ok) return true;
  }
  return false;
}
// Largest K/V volume of a launch whose tile loads carry the L2 "evict first" hint (see ptenc_attn_kv_hint).
#ifndef PTENC_ATTN_EVICT_FIRST_MAX_BYTES
#define PTENC_ATTN_EVICT_FIRST_MAX_BYTES (4ull << 30)
#endif
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// hinted != 0: the copy carries the L2 eviction policy `pol`
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar,
                                            int hinted, uint64_t pol) {
  if (hinted) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(pol) : "memory");
  } else {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
  }
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8) += A(16x16) B(16x8), all sixteen rows in use.
__device__ __forceinline__ void mma_full(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Transposes an 8x8 matrix of 16-bit values held one row pair per lane across the warp.
__device__ __forceinline__ uint32_t movm_t(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void consumer_sync(int nthreads) {
  asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

// ------------------------------------------------------------------------------------------------ schedule
// Tiles of one ring that hold live slots.  Live slots are the pinned entries [0, sink) and the `count` slots of the
// sliding part, which starts at slot sink + head and wraps inside [sink, W).  As a set of slots that is a low
// interval [0, end1) (pinned entries plus the wrapped tail of the sliding part) and a high interval starting at
// sink + head.  The unit's tiles are enumerated high interval first: tile t0 + i for i < len2, then tile i - len2.
template <int TILE_N>
__device__ __forceinline__ int live_tiles(int sink, int head, int count, int W, int* t0, int* len2) {
  int end1 = sink, n2 = 0;
  if (count > 0) {
    const int first = (W - sink) - head;            // sliding slots before the wrap
    if (count > first) { end1 = sink + (count - first); n2 = first; } else n2 = count;
  }
  const int e1 = end1 > 0 ? (end1 - 1) / TILE_N : -1;
  if (n2 == 0) { *t0 = 0; *len2 = 0; return e1 + 1; }
  const int s2 = sink + head;
  const int t2 = s2 / TILE_N, e2 = (s2 + n2 - 1) / TILE_N;
  *t0 = t2;
  *len2 = e2 - t2 + 1;
  const int low = (e1 + 1) < t2 ? (e1 + 1) : t2;    // low-interval tiles not already counted in the high run
  return *len2 + low;
}

struct Entry {          // one (layer, sequence) of the call
  int head, count, sink, nt, t0, len2;
};

template <int D, int TILE_N, int NW, int STAGES>
struct Smem {
  static_assert(STAGES % NW == 0, "a stage must always be consumed by the same warp");
  static_assert(TILE_N % 16 == 0 && (D == 64 || D == 128), "tile shape");
  static constexpr int K_BYTES = TILE_N * D * 2;
  static constexpr int STAGE_BYTES = 2 * K_BYTES;
  static constexpr int Q_BYTES = 8 * D * 2;
  static constexpr int ACC_STRIDE = D + 8;
  static constexpr int OFF_Q = STAGES * STAGE_BYTES;
  static constexpr int OFF_ACC = OFF_Q + 2 * Q_BYTES;
  static constexpr int OFF_ML = OFF_ACC + NW * 8 * ACC_STRIDE * 4;
  static constexpr int OFF_BAR = OFF_ML + NW * 16 * 4;
  static constexpr int OFF_MISC = OFF_BAR + (2 * STAGES + 4) * 8;
  static constexpr int OFF_DESC = OFF_MISC + 64;            // two work-item descriptions of 16 ints
  static constexpr int TOTAL = OFF_DESC + 128;
};

// ------------------------------------------------------------------------------------------------ kernel
// SCORE: the cache runs the importance-aware eviction policy.  Live slots are then given by a bitmap instead of a
// ring interval, and the launch leaves behind what the policy needs to turn this attention into per-token mass: the
// scaled logits of every live slot (base-2 domain, [unit][slot][8 heads]) and the log2-sum-exp2 of every query head.
template <int D, int TILE_N, int NW, int STAGES, bool SCORE>
__global__ void __launch_bounds__((NW + 1 + PTENC_ATTN_ENC_WARPS) * 32, PTENC_ATTN_CTAS_PER_SM)
k_attn_bf16(const PtencDev p, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
            const int l0, const int nl, const __nv_bfloat16* __restrict__ q, const uint8_t* __restrict__ active,
            __nv_bfloat16* __restrict__ out, float* __restrict__ lse, const int fold_staged, const int kv_hint) {
  using SM = Smem<D, TILE_N, NW, STAGES>;
  constexpr int NE = PTENC_ATTN_ENC_WARPS;
  constexpr int NTHREADS = (NW + 1 + NE) * 32;               // consumers, the TMA producer, the encoder warps
  constexpr int NCONS = NW * 32;
  constexpr int KSTEPS = D / 16;
  constexpr int HALF_BYTES = TILE_N * 128;     // one 64-column half of a tile

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  float* mb_acc = reinterpret_cast<float*>(smem + SM::OFF_ACC);
  float* mb_ml = reinterpret_cast<float*>(smem + SM::OFF_ML);
  const uint32_t bar_full = smem_base + SM::OFF_BAR;
  const uint32_t bar_empty = bar_full + STAGES * 8;
  const uint32_t bar_qfull = bar_empty + STAGES * 8;
  const uint32_t bar_qempty = bar_qfull + 2 * 8;
  volatile int* misc = reinterpret_cast<volatile int*>(smem + SM::OFF_MISC);
  // misc[0] abort flag, misc[1] last-arriver flag, misc[8..9] verdict on the item in description slot 0 / 1
  // (1 = work on it, 2 = stop)
  volatile int* desc = reinterpret_cast<volatile int*>(smem + SM::OFF_DESC);
  // description of a work item: [0] 1 = item, 2 = no more items; [1] layer of the call, [2] sequence, [3] KV head;
  // [4..8] ring state and tile enumeration of the unit (head, count, pinned, t0, len2); [9] first tile of the piece
  // in the unit's enumeration, [10] tiles of the piece; [11] pieces of the unit, [12] this piece, [13] first partial
  // slot of the unit (split units only)
  __shared__ long long s_part[NTHREADS / 32];
  __shared__ int s_items[NTHREADS + 1];
  __shared__ int s_split[NTHREADS + 1];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int W = p.W, B = p.B, Hkv = p.Hkv, g = p.g;
  const int n_t = (W + TILE_N - 1) / TILE_N;
  const int n_ent = nl * B;

  // ---- set-up: barriers, zero padding rows of the Q buffers ---------------------------------------
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(bar_qfull + 8 * s, 1); mbar_init(bar_qempty + 8 * s, NW); }
    misc[0] = 0; misc[1] = 0; misc[8] = 0; misc[9] = 0;
    desc[0] = 0; desc[16] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid == NW * 32) {                                      // the two tensor maps are wanted at the first tile
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmK)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmV)) : "memory");
  }
  for (int i = tid; i < 2 * SM::Q_BYTES / 4; i += NTHREADS) reinterpret_cast<uint32_t*>(smem + SM::OFF_Q)[i] = 0u;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  // When the launch was allowed to start before the kernel in front of it on the stream has finished (the fused
  // step does that with its append/evict kernel), everything up to here overlapped that kernel; nothing it wrote is
  // read before this point.  A no-op for an ordinary launch.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- schedule ----------------------------------------------------------------------------------------------------
  // Work items.  The tiles of a (layer, sequence, KV head) unit are one item, or -- when the call has too few tiles
  // to give every CTA several items -- P pieces of about `piece` tiles each.  Items are numbered in (entry, head,
  // piece) order and handed out at run time: a CTA that finishes an item takes the next number from a counter in
  // global memory.  SMs do not all stream at the same rate (a fixed equal share left the slowest of them 10 % behind
  // the median at the largest shapes), so the hand-out is dynamic; which CTA computes an item has no influence on
  // the result.
  struct Raw { int head, count, sink, act; long long n; };
  // the ring words of one entry; every load is unconditional (index clamped) so that the loads of several entries
  // can be in flight together
  auto fetch = [&](int e) -> Raw {
    Raw r;
    const int ec = e < 0 ? 0 : (e >= n_ent ? n_ent - 1 : e);
    const int li = ec / B, b = ec - li * B;
    const size_t lb = (size_t)(l0 + li) * B + b;
    r.act = (active != nullptr) ? (int)active[b] : 1;
    r.sink = p.n_sink != nullptr ? p.n_sink[lb] : 0;
    r.head = SCORE ? 0 : p.head[lb];
    r.count = SCORE ? 0 : p.count[lb];
    r.n = SCORE ? p.n_app[lb] : 0;
    return r;
  };
  auto make_entry = [&](const Raw& r, int e) -> Entry {
    Entry en;
    en.head = en.count = en.sink = en.nt = en.t0 = en.len2 = 0;
    if (e < 0 || e >= n_ent || r.act == 0) return en;            // out of range or inactive: no tiles
    en.sink = r.sink;
    if (SCORE) {
      // slots fill in order until the window is full and are reused in place afterwards: the slots in use are a
      // prefix [0, min(n_appended, W)); which of them hold a token is the bitmap's business (see the mask below)
      en.head = 0;
      en.count = (int)(r.n < (long long)W ? r.n : (long long)W) - en.sink;
    } else {
      en.head = r.head;
      en.count = r.count;
    }
    const int cap = W - en.sink;
    if (en.sink < 0 || cap < 1 || en.head < 0 || en.head >= cap || en.count < 0 || en.count > cap) {
      // a ring state outside its range (corrupt workspace, or bad head/count arrays handed to the static-scratch
      // entry): the sequence is skipped, nothing of it is loaded, and the status word says so
      atomicOr(p.status, PTENC_ST_BAD_INDEX);
      en.head = en.count = en.sink = 0;
      return en;
    }
    en.nt = live_tiles<TILE_N>(en.sink, en.head, en.count, W, &en.t0, &en.len2);
    return en;
  };
  auto load_entry = [&](int e) -> Entry { return make_entry(fetch(e), e); };
  // every thread takes a contiguous chunk of the entries; tiles, items and pieces of split units per chunk.  This
  // code runs once per launch, straight from instruction memory that the K/V stream of the launch before has pushed
  // out of every cache: it is kept short (rolled loops, sums and prefixes through warp shuffles), and the second
  // pass over the entries is skipped when no unit is split, which the first pass can tell.
  const int chunk = (n_ent + NTHREADS - 1) / NTHREADS;
  const int e_lo = min(tid * chunk, n_ent), e_hi = min(e_lo + chunk, n_ent);
  constexpr int NWARPS = NTHREADS / 32;
  // In the common launch -- every entry has tiles and no unit is split -- item i is simply (entry i / H_kv, head
  // i % H_kv), and CTA c starts on item c: the ring words of that entry are requested now, with the first pass.
  const Raw first_raw = fetch((int)blockIdx.x / Hkv);
  // The producer's first request to the work counter (the number of its second item, or its one failing grab) is
  // made here as well, so that the answer is there when the first item's tiles have been issued.
  int first_grab = 0;
  if (tid == NW * 32) first_grab = atomicAdd(p.work, 1) + (int)gridDim.x;
  long long mine = 0;
  int nz = 0, mx = 0;                                        // entries with tiles, longest entry
#pragma unroll 1
  for (int e = e_lo; e < e_hi; e += 4) {                      // four entries' ring words requested at once
    Raw r[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) r[u] = fetch(e + u < e_hi ? e + u : e_hi - 1);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (e + u < e_hi) {
        const int nt = make_entry(r[u], e + u).nt;
        mine += nt;
        nz += nt > 0 ? 1 : 0;
        mx = max(mx, nt);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mine += __shfl_xor_sync(0xffffffffu, mine, o);
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  __shared__ int s_wsum[3][NWARPS];
  if (lane == 0) { s_part[warp] = mine; s_wsum[2][warp] = mx; }
  __syncthreads();
  long long total = 0;
  int longest = 0;
#pragma unroll
  for (int i = 0; i < NWARPS; ++i) { total += s_part[i]; longest = max(longest, s_wsum[2][i]); }
  const long long T = total * Hkv;                     // tiles of the whole call
  // piece size: about `bal` items per CTA when the call is small; a unit is never cut finer than 8 tiles.  With
  // bal <= part_slots / (2 gridDim) the pieces of split units always fit the partial slots: a unit is split only if
  // it has more than `piece` tiles, so there are at most T / piece + T / piece <= 2 bal gridDim such pieces.
  long long bal = p.part_slots / (2 * (long long)gridDim.x);
  bal = bal < 1 ? 1 : (bal > 4 ? 4 : bal);
  long long piece_ll = (T + bal * gridDim.x - 1) / (bal * gridDim.x);
  const int piece = (int)(piece_ll < 8 ? 8 : (piece_ll > (1 << 24) ? (1 << 24) : piece_ll));
  auto pieces_of = [&](int nt) -> int { return nt <= 0 ? 0 : (nt + piece - 1) / piece; };
  {
    int items = Hkv * nz, split = 0;                          // no unit longer than a piece: every unit is one item
    if (longest > piece) {                                    // uniform over the CTA
      items = 0;
#pragma unroll 1
      for (int e = e_lo; e < e_hi; ++e) {                     // the ring words are in L1 or L2 now
        const int pc = pieces_of(load_entry(e).nt);
        items += Hkv * pc;
        if (pc > 1) split += Hkv * pc;
      }
    }
    // exclusive prefixes over the threads: inclusive scan inside the warp, then the warps' totals
    int ci = items, cs = split;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, ci, o), c = __shfl_up_sync(0xffffffffu, cs, o);
      if (lane >= o) { ci += a; cs += c; }
    }
    if (lane == 31) { s_wsum[0][warp] = ci; s_wsum[1][warp] = cs; }
    __syncthreads();
    int bi = ci - items, bs = cs - split, ti = 0, ts = 0;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) {
      if (w < warp) { bi += s_wsum[0][w]; bs += s_wsum[1][w]; }
      ti += s_wsum[0][w]; ts += s_wsum[1][w];
    }
    s_items[tid] = bi;                                        // exclusive prefixes; the totals go last
    s_split[tid] = bs;
    if (tid == 0) { s_items[NTHREADS] = ti; s_split[NTHREADS] = ts; }
  }
  __syncthreads();
  const int n_items = s_items[NTHREADS];
  const bool plain = longest <= piece && n_items == Hkv * n_ent;   // see above; uniform over the launch

  if (warp > NW) {
    // ================================================================ encoder warps (see the file header)
    // (layer, sequence) pairs of the call, dealt round-robin to the encoder warps of all CTAs; they take no part in
    // anything below.  Under the K/V stream a dependent memory round trip takes microseconds, and a pair is a chain
    // of about a dozen: several warps per CTA keep the chain off the critical path at any batch size.
    if (fold_staged && p.encode_enabled) {
      for (int e = blockIdx.x * NE + (warp - NW - 1); e < n_ent; e += gridDim.x * NE) {
        const int li = e / B, b = e - li * B;
        const int l = l0 + li;
        const size_t lb = (size_t)l * B + b;
        if (!p.enc_set[l] || p.n_staged[lb] <= 0) continue;
        if (active != nullptr && active[b] == 0) continue;
        encw_fold_row(p, l, lb, reinterpret_cast<const __nv_bfloat16*>(p.stageK) + lb * p.d_kv,
                      reinterpret_cast<const __nv_bfloat16*>(p.stageV) + lb * p.d_kv, lane);
      }
    }
    return;
  }

  const float sl2 = 1.4426950408889634f / sqrtf((float)D);
  // Pipeline stages belong to consumer warps: warp w owns stages [w SPW, (w + 1) SPW) and takes the tiles i = w
  // (mod NW) of every item, so a stage's barriers always have the same consumer, and which warp sums which tiles of
  // an item does not depend on what the CTA worked on before (results are reproducible bit for bit).
  constexpr int SPW = STAGES / NW;

  if (warp == NW) {
    // ================================================================ producer warp
    // All lanes look an item up (ballots and scans over the chunk prefixes); lane 0 posts the item's description and
    // its Q rows; lane w < NW feeds consumer warp w: it issues the tiles i = w (mod NW) of every item into that warp's
    // stages.  One lane issuing every tile of the CTA (a barrier wait, the transaction count and four bulk copies
    // per tile, ~0.3 us) could just keep up with one SM's share of the HBM stream and fell behind at every item
    // boundary; NW lanes in parallel have headroom.
    const uint64_t kv_policy = l2_evict_first_policy();
    uint32_t kmine = 0;                                      // tiles this lane has issued into its warp's stages
    uint32_t useq = 0;                                       // items handed to the consumers
    bool aborted = false;
    const long long rows_total = (long long)p.L * B * Hkv * W;

    // Looking an item up (which entry, head and piece it is) needs the ring words of up to 32 entries, and with
    // nearly all of the SM's memory used as shared memory those loads miss L1: a round trip through L2 that takes
    // microseconds under the K/V stream.  So the look-up is split: `begin` finds the chunk of entries and requests
    // their ring words, `finish` uses them -- and between the two the tiles of the item before are issued.  The
    // number of an item is requested from the global counter one step earlier still.
    struct Item { int kind, e, h, k, iu_lo, n_mine, P, slot_base; Entry en; };     // kind 0 bad, 1 item, 2 none left
    struct Pending { int item, tch, ce_lo, ce_hi; Raw raw; };
    auto lookup_begin = [&](int item) -> Pending {
      Pending pd;
      pd.item = item; pd.tch = -1; pd.ce_lo = pd.ce_hi = 0;
      pd.raw.head = pd.raw.count = pd.raw.sink = pd.raw.act = 0; pd.raw.n = 0;
      if (item >= n_items) return pd;
      if (plain) {                                           // no search: the entry follows from the item's number
        pd.tch = -2;
        pd.ce_lo = item / Hkv;
        pd.raw = fetch(pd.ce_lo);
        return pd;
      }
      for (int base = 0; base < NTHREADS; base += 32) {
        const int idx = base + lane;
        const bool hit = idx < NTHREADS && s_items[idx] <= item && item < s_items[idx + 1];
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (m != 0) { pd.tch = base + __ffs(m) - 1; break; }
      }
      if (pd.tch >= 0) {
        pd.ce_lo = min(pd.tch * chunk, n_ent);
        pd.ce_hi = min(pd.ce_lo + chunk, n_ent);
        pd.raw = fetch(pd.ce_lo + lane);                     // the first 32 entries of the chunk; clamped, unconditional
      }
      return pd;
    };
    auto lookup_finish = [&](const Pending& pd) -> Item {
      Item it;
      it.kind = 0; it.e = -1; it.h = it.k = it.iu_lo = it.n_mine = it.P = it.slot_base = 0;
      it.en.head = it.en.count = it.en.sink = it.en.nt = it.en.t0 = it.en.len2 = 0;
      if (pd.item >= n_items) { it.kind = 2; return it; }
      if (pd.tch == -2) {
        it.e = pd.ce_lo;
        it.en = make_entry(pd.raw, it.e);
        it.h = pd.item - it.e * Hkv;
        it.P = 1;
        it.n_mine = it.en.nt;
        if (it.n_mine > 0) it.kind = 1;
        return it;
      }
      if (pd.tch < 0) return it;
      int rem = pd.item - s_items[pd.tch];
      int split_before = s_split[pd.tch];
      for (int base = pd.ce_lo; base < pd.ce_hi && it.e < 0; base += 32) {
        const int ee = base + lane;
        const Entry le = (ee >= pd.ce_hi) ? make_entry(pd.raw, -1)
                                          : (base == pd.ce_lo ? make_entry(pd.raw, ee) : load_entry(ee));
        const int pc = pieces_of(le.nt);
        const int cnt = Hkv * pc, sp = pc > 1 ? cnt : 0;
        int c_inc = cnt, s_inc = sp;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int a = __shfl_up_sync(0xffffffffu, c_inc, o), c = __shfl_up_sync(0xffffffffu, s_inc, o);
          if (lane >= o) { c_inc += a; s_inc += c; }
        }
        const bool hit = cnt > 0 && c_inc - cnt <= rem && rem < c_inc;
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (m != 0) {
          const int src = __ffs(m) - 1;
          it.e = base + src;
          rem -= __shfl_sync(0xffffffffu, c_inc - cnt, src);
          split_before += __shfl_sync(0xffffffffu, s_inc - sp, src);
          it.en.head = __shfl_sync(0xffffffffu, le.head, src);
          it.en.count = __shfl_sync(0xffffffffu, le.count, src);
          it.en.sink = __shfl_sync(0xffffffffu, le.sink, src);
          it.en.nt = __shfl_sync(0xffffffffu, le.nt, src);
          it.en.t0 = __shfl_sync(0xffffffffu, le.t0, src);
          it.en.len2 = __shfl_sync(0xffffffffu, le.len2, src);
        } else {
          rem -= __shfl_sync(0xffffffffu, c_inc, 31);
          split_before += __shfl_sync(0xffffffffu, s_inc, 31);
        }
      }
      it.P = pieces_of(it.en.nt);
      if (it.e < 0 || it.P <= 0 || rem < 0 || rem >= Hkv * it.P) return it;
      it.h = rem / it.P;
      it.k = rem - it.h * it.P;
      it.iu_lo = (int)((long long)it.k * it.en.nt / it.P);
      it.n_mine = (int)((long long)(it.k + 1) * it.en.nt / it.P) - it.iu_lo;
      it.slot_base = it.P > 1 ? split_before + it.h * it.P : 0;
      if (it.n_mine <= 0 || it.slot_base + it.P > p.part_slots) return it;
      it.kind = 1;
      return it;
    };
    // Item numbers: CTA c starts on item c without asking; the counter hands out gridDim.x, gridDim.x + 1, ...
    auto grab = [&]() -> int { return lane == 0 ? atomicAdd(p.work, 1) + (int)gridDim.x : 0; };
    const int last_grab = max(n_items, (int)gridDim.x) + (int)gridDim.x - 1;   // what the launch's last grab returns

    Pending pd;
    if (plain && (int)blockIdx.x < n_items) {                // the first item's ring words are here already
      pd.item = (int)blockIdx.x; pd.tch = -2; pd.ce_lo = (int)blockIdx.x / Hkv; pd.ce_hi = 0;
      pd.raw = first_raw;
    } else {
      pd = lookup_begin((int)blockIdx.x);
    }
    int grabbed = first_grab;                                // the item after that; every CTA makes exactly one grab
                                                             // that finds nothing left (this one, if it has no item)
    while (!aborted) {
      const Item cur = lookup_finish(pd);
      const uint32_t ubuf = useq & 1;
      volatile int* dsc = desc + ubuf * 16;
      if (cur.kind != 1) {
        if (cur.kind == 0) {                                 // uniform over the warp
          if (lane == 0) atomicOr(p.status, PTENC_ST_BAD_SCHEDULE);
          aborted = true;
          break;
        }
        // nothing left: tell the consumers, and the CTA whose grab was the very last of the launch rewinds the counter
        if (lane == 0) {
          if (grabbed == last_grab) *p.work = 0;
          if (mbar_wait(bar_qempty + 8 * ubuf, ((useq >> 1) & 1) ^ 1)) {
            dsc[0] = 2;
            mbar_arrive(bar_qfull + 8 * ubuf);
          } else {
            aborted = true;
          }
        }
        break;
      }
      const int e = cur.e, h = cur.h, n_mine = cur.n_mine, iu_lo = cur.iu_lo;
      const Entry en = cur.en;
      const int li = e / B, b = e - li * B;
      if (lane == 0) {
        // the item's description and the Q rows of its unit
        if (!mbar_wait(bar_qempty + 8 * ubuf, ((useq >> 1) & 1) ^ 1)) { aborted = true; }
        if (!aborted) {
          dsc[1] = li; dsc[2] = b; dsc[3] = h; dsc[4] = en.head; dsc[5] = en.count; dsc[6] = en.sink;
          dsc[7] = en.t0; dsc[8] = en.len2; dsc[9] = iu_lo; dsc[10] = n_mine; dsc[11] = cur.P; dsc[12] = cur.k;
          dsc[13] = cur.slot_base; dsc[0] = 1;
          const uint32_t qbytes = (uint32_t)(g * D * 2);
          mbar_expect_tx(bar_qfull + 8 * ubuf, qbytes);
          bulk_load(smem_base + SM::OFF_Q + ubuf * SM::Q_BYTES,
                    q + (((size_t)li * B + b) * p.Hq + (size_t)h * g) * D, qbytes, bar_qfull + 8 * ubuf);
        }
      }
      // the next item: its number has arrived by now; request its entries' ring words, and the number after it
      const int item2 = __shfl_sync(0xffffffffu, grabbed, 0);
      pd = lookup_begin(item2);
      if (item2 < n_items) grabbed = grab();
      aborted = __shfl_sync(0xffffffffu, aborted ? 1 : 0, 0) != 0;
      if (lane < NW && !aborted) {
        const size_t lb = (size_t)(l0 + li) * B + b;
        const long long row0 = ((long long)lb * Hkv + h) * W;
        for (int i = lane; i < n_mine; i += NW) {
          const int iu = iu_lo + i;                          // tile of the unit, in its enumeration order
          const int j = iu < en.len2 ? en.t0 + iu : iu - en.len2;
          const uint32_t s = lane * SPW + kmine % SPW;
          const long long yy = row0 + (long long)j * TILE_N;
          if (j < 0 || j >= n_t || yy < 0 || yy >= rows_total) {
            atomicOr(p.status, PTENC_ST_BAD_INDEX); aborted = true; break;
          }
          if (!mbar_wait(bar_empty + 8 * s, ((kmine / SPW) & 1) ^ 1)) { aborted = true; break; }
          const uint32_t dst = smem_base + s * SM::STAGE_BYTES;
          const uint32_t fb = bar_full + 8 * s;
          mbar_expect_tx(fb, SM::STAGE_BYTES);
          const int y = (int)yy;
#pragma unroll
          for (int hf = 0; hf < D / 64; ++hf) {
            tma_load_2d(dst + hf * HALF_BYTES, &tmK, hf * 64, y, fb, kv_hint, kv_policy);
            tma_load_2d(dst + SM::K_BYTES + hf * HALF_BYTES, &tmV, hf * 64, y, fb, kv_hint, kv_policy);
          }
          kmine += 1;
        }
      }
      aborted = __any_sync(0xffffffffu, aborted);
      ++useq;
    }
    aborted = __any_sync(0xffffffffu, aborted);
    if (aborted) {
      if (lane == 0) { atomicOr(p.status, PTENC_ST_WAIT_TIMEOUT); misc[0] = 1; }
      // copies still in flight must land before the CTA's shared memory goes away
      if (lane < NW) {
        const uint32_t back = kmine < (uint32_t)SPW ? kmine : (uint32_t)SPW;
        for (uint32_t i = 0; i < back; ++i) {
          const uint32_t kk = kmine - 1 - i;
          (void)mbar_wait(bar_full + 8 * (lane * SPW + kk % SPW), (kk / SPW) & 1);
        }
      }
    }
    return;
  }

  // ================================================================== consumer warps
  const int qr = lane >> 2;          // row of the fragment = query head within the group
  const int qc = lane & 3;
  uint32_t kq = 0;                   // tiles this warp has consumed
  uint32_t useq = 0;
  // The next item is announced by one thread: it waits for the item's barrier and posts a verdict that everybody reads
  // behind a consumer barrier, so that the warps agree on going on or stopping even when a wait runs out.
  auto announce = [&](uint32_t us) {
    const uint32_t ub2 = us & 1;
    int v = 2;
    if (misc[0] == 0 && mbar_wait(bar_qfull + 8 * ub2, (us >> 1) & 1)) v = desc[ub2 * 16];
    else { atomicOr(p.status, PTENC_ST_WAIT_TIMEOUT); misc[0] = 1; }
    misc[8 + ub2] = v;
  };
  if (tid == 0) announce(0);
  consumer_sync(NCONS);

  while (true) {
    const uint32_t ubuf = useq & 1;
    if (misc[8 + ubuf] != 1) break;                          // no more items (or a wait ran out): uniform over the CTA
    (void)mbar_wait(bar_qfull + 8 * ubuf, (useq >> 1) & 1);  // completed already; orders this thread's reads behind it
    volatile int* dsc = desc + ubuf * 16;
    const int li = dsc[1], b = dsc[2], h = dsc[3];
    const int head = dsc[4], count = dsc[5], sink = dsc[6], t0 = dsc[7], len2 = dsc[8];
    const int iu_lo = dsc[9], n_mine = dsc[10], n_parts = dsc[11], piece_k = dsc[12], slot_base = dsc[13];
    const int cap = W - sink;

    // ---- Q fragments (A operand, rows = heads; rows >= g are zero) ------------------------------------
    uint32_t qa[KSTEPS][2];
    {
      const uint8_t* qb = smem + SM::OFF_Q + ubuf * SM::Q_BYTES + qr * (D * 2) + qc * 4;
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        qa[ks][0] = *reinterpret_cast<const uint32_t*>(qb + ks * 32);
        qa[ks][1] = *reinterpret_cast<const uint32_t*>(qb + ks * 32 + 16);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_qempty + 8 * ubuf);     // the description and the Q rows have been read
    }

    // Transposed products, so that the 16 rows of the mma are always full: S^T = K Q^T (rows = tokens, columns = the
    // query heads) and O^T += V^T P^T (rows = head dims, columns = heads).  A lane (qr, qc) then owns the two heads
    // 2 qc and 2 qc + 1: their running maxima and sums, and the columns of O^T that belong to them.
    constexpr int MT = TILE_N / 16;                // 16-token row tiles of S^T = k-steps of the second product
    constexpr int DT = D / 16;                     // 16-dim row tiles of O^T
    float m_run0 = -INFINITY, m_run1 = -INFINITY, l_run0 = 0.f, l_run1 = 0.f;
    float oT[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i) { oT[i][0] = 0.f; oT[i][1] = 0.f; oT[i][2] = 0.f; oT[i][3] = 0.f; }

    for (int i = warp; i < n_mine; i += NW, ++kq) {
      const uint32_t s = warp * SPW + kq % SPW;
      const int iu = iu_lo + i;
      const int j = iu < len2 ? t0 + iu : iu - len2;
      uint32_t lw0 = 0xffffffffu, lw1 = 0xffffffffu;        // liveness of the tile's slots (SCORE), requested early
      if (SCORE) {
        const unsigned int* lw = p.live_bits + ((size_t)(l0 + li) * B + b) * p.wb + ((j * TILE_N) >> 5);
        lw0 = lw[0];
        if (TILE_N > 32) lw1 = lw[1];
      }
      if (misc[0] == 0 && !mbar_wait(bar_full + 8 * s, (kq / SPW) & 1)) {
        atomicOr(p.status, PTENC_ST_WAIT_TIMEOUT);
        misc[0] = 1;
      }
      __syncwarp();
      const uint32_t kb = smem_base + s * SM::STAGE_BYTES;
      const uint32_t vb = kb + SM::K_BYTES;

      // ---- S^T = K Q^T: A = a 16-token x 16-dim block of K (ldmatrix), B = the Q fragments ----------------------
      float sT[MT][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) { sT[mt][0] = 0.f; sT[mt][1] = 0.f; sT[mt][2] = 0.f; sT[mt][3] = 0.f; }
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        const int cidx = 2 * ks + (lane >> 4);               // 16-byte chunk of the row
        const int hf = cidx >> 3, cc = cidx & 7;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const int row = 16 * mt + (lane & 7) + ((lane >> 3) & 1) * 8;
          uint32_t a0, a1, a2, a3;
          ldsm_x4(kb + hf * HALF_BYTES + row * 128 + ((cc ^ (row & 7)) << 4), a0, a1, a2, a3);
          mma_full(sT[mt], a0, a1, a2, a3, qa[ks][0], qa[ks][1]);
        }
      }
      // ---- mask slots that hold no live token (rows qr and qr + 8 of each row tile) -------------------------------
      const int slot0 = j * TILE_N;
      if (SCORE) {
        if ((lw0 & lw1) != 0xffffffffu) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              const int o = 16 * mt + qr + 8 * x;               // slot within the tile
              const bool live = (((o < 32 ? lw0 : lw1) >> (o & 31)) & 1u) != 0;
              if (!live) { sT[mt][2 * x] = -INFINITY; sT[mt][2 * x + 1] = -INFINITY; }
            }
          }
        }
        // scaled logits of the live slots: a lane holds heads 2 qc, 2 qc + 1 of tokens qr and qr + 8 of each row tile
        float* lg = p.logits + ((((size_t)(l0 + li) * B + b) * Hkv + h) * W + slot0) * 8 + 2 * qc;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            const int o = 16 * mt + qr + 8 * x;
            if (sT[mt][2 * x] != -INFINITY && slot0 + o < W)
              *reinterpret_cast<float2*>(lg + (size_t)o * 8) = make_float2(sT[mt][2 * x] * sl2, sT[mt][2 * x + 1] * sl2);
          }
        }
      } else {
        bool full = false;
        if (slot0 + TILE_N <= sink) {
          full = true;
        } else if (slot0 >= sink && slot0 + TILE_N <= W) {
          int d0 = slot0 - sink - head;
          if (d0 < 0) d0 += cap;
          full = (count == cap) || (d0 + TILE_N <= count);
        }
        if (!full) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              const int slot = slot0 + 16 * mt + qr + 8 * x;
              int dd = slot - sink - head;
              if (dd < 0) dd += cap;
              const bool live = slot < sink || (slot < W && dd < count);
              if (!live) { sT[mt][2 * x] = -INFINITY; sT[mt][2 * x + 1] = -INFINITY; }
            }
          }
        }
      }
      // ---- online softmax (base 2), two heads per lane, reduced over the eight token rows of the lanes ----------
      float mx0 = sT[0][0], mx1 = sT[0][1];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        mx0 = fmaxf(mx0, fmaxf(sT[mt][0], sT[mt][2]));
        mx1 = fmaxf(mx1, fmaxf(sT[mt][1], sT[mt][3]));
      }
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
      }
      const float m_new0 = fmaxf(m_run0, mx0 * sl2), m_new1 = fmaxf(m_run1, mx1 * sl2);
      const float m_use0 = (m_new0 == -INFINITY) ? 0.f : m_new0;     // all-masked: keep exp2 arguments finite
      const float m_use1 = (m_new1 == -INFINITY) ? 0.f : m_new1;
      const float corr0 = ex2(m_run0 - m_use0), corr1 = ex2(m_run1 - m_use1);
      float psum0 = 0.f, psum1 = 0.f;
      uint32_t pb[MT][2];                                    // P^T as B fragments: [tokens 2qc.., +8][head qr]
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const float p00 = ex2(fmaf(sT[mt][0], sl2, -m_use0));      // token qr,     head 2qc
        const float p01 = ex2(fmaf(sT[mt][1], sl2, -m_use1));      // token qr,     head 2qc + 1
        const float p10 = ex2(fmaf(sT[mt][2], sl2, -m_use0));      // token qr + 8, head 2qc
        const float p11 = ex2(fmaf(sT[mt][3], sl2, -m_use1));
        psum0 += p00 + p10;
        psum1 += p01 + p11;
        pb[mt][0] = movm_t(pack_bf16(p00, p01));             // 8 x 8 transpose across the warp
        pb[mt][1] = movm_t(pack_bf16(p10, p11));
      }
      l_run0 = l_run0 * corr0 + psum0;
      l_run1 = l_run1 * corr1 + psum1;
      m_run0 = m_new0;
      m_run1 = m_new1;
      if (__any_sync(0xffffffffu, corr0 != 1.f || corr1 != 1.f)) {
#pragma unroll
        for (int dt = 0; dt < DT; ++dt) { oT[dt][0] *= corr0; oT[dt][1] *= corr1; oT[dt][2] *= corr0; oT[dt][3] *= corr1; }
      }
      // ---- O^T += V^T P^T: A = a 16-dim x 16-token block of V^T (ldmatrix.trans), B = P^T ------------------------
#pragma unroll
      for (int kt = 0; kt < MT; ++kt) {
        const int row = 16 * kt + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int dt = 0; dt < DT; ++dt) {
          const int cidx = 2 * dt + (lane >> 4);
          const int hf = cidx >> 3, cc = cidx & 7;
          uint32_t r0, r1, r2, r3;           // (tok 0-7, d 0-7), (tok 8-15, d 0-7), (tok 0-7, d 8-15), (tok 8-15, d 8-15)
          ldsm_x4_t(vb + hf * HALF_BYTES + row * 128 + ((cc ^ (row & 7)) << 4), r0, r1, r2, r3);
          mma_full(oT[dt], r0, r2, r1, r3, pb[kt][0], pb[kt][1]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * s);
    }

    // ---- the warp's partials of this unit -> shared memory ---------------------------------------------------------
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      l_run0 += __shfl_xor_sync(0xffffffffu, l_run0, o);
      l_run1 += __shfl_xor_sync(0xffffffffu, l_run1, o);
    }
    {
      float* acc0 = mb_acc + (warp * 8 + 2 * qc) * SM::ACC_STRIDE + qr;      // head 2 qc, dim qr (+ 8, + 16 dt)
      float* acc1 = acc0 + SM::ACC_STRIDE;                                    // head 2 qc + 1
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
        acc0[16 * dt] = oT[dt][0];
        acc1[16 * dt] = oT[dt][1];
        acc0[16 * dt + 8] = oT[dt][2];
        acc1[16 * dt + 8] = oT[dt][3];
      }
      if (qr == 0) {
        mb_ml[warp * 16 + 2 * qc] = m_run0;
        mb_ml[warp * 16 + 2 * qc + 1] = m_run1;
        mb_ml[warp * 16 + 8 + 2 * qc] = l_run0;
        mb_ml[warp * 16 + 8 + 2 * qc + 1] = l_run1;
      }
    }
    consumer_sync(NCONS);

    const bool whole = n_parts == 1;
    const size_t unit_id = ((size_t)(l0 + li) * B + b) * Hkv + h;
    const size_t orow0 = ((size_t)li * B + b) * p.Hq + (size_t)h * g;
    const int my_slot = slot_base + piece_k;                  // used by pieces of split units only
    if (h < 0 || h >= Hkv || n_mine <= 0 || n_parts < 1 || (!whole && slot_base + n_parts > p.part_slots)) {
      if (tid == 0) { atomicOr(p.status, PTENC_ST_BAD_SCHEDULE); announce(useq + 1); }   // uniform over the CTA
      consumer_sync(NCONS);
      ++useq;
      continue;
    }

    // NCONS / 8 threads per query-head row: the row's merge weights are computed once per thread
    {
      constexpr int TPR = NCONS / 8;
      const int r = tid / TPR, d0 = tid - r * TPR;
      float mt = -INFINITY;
#pragma unroll
      for (int w = 0; w < NW; ++w) mt = fmaxf(mt, mb_ml[w * 16 + r]);
      float wg[NW];
      float lt = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float mw = mb_ml[w * 16 + r];
        wg[w] = (mw == -INFINITY) ? 0.f : ex2(mw - mt);
        lt = fmaf(wg[w], mb_ml[w * 16 + 8 + r], lt);
      }
      if (whole) {
        if (r < g) {
#pragma unroll
          for (int d = d0; d < D; d += TPR) {
            float acc = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) acc = fmaf(wg[w], mb_acc[(w * 8 + r) * SM::ACC_STRIDE + d], acc);
            out[(orow0 + r) * D + d] = __float2bfloat16_rn(acc / lt);
          }
          if (lse != nullptr && d0 == 0) lse[orow0 + r] = (mt + log2f(lt)) * 0.6931471805599453f;
          if (SCORE && d0 == 0) p.lse2[((size_t)(l0 + li) * B + b) * p.Hq + (size_t)h * g + r] = mt + log2f(lt);
        }
        if (SCORE && tid == 0) p.pending[(size_t)(l0 + li) * B + b] = 1;
      } else {
#pragma unroll
        for (int d = d0; d < D; d += TPR) {
          float acc = 0.f;
#pragma unroll
          for (int w = 0; w < NW; ++w) acc = fmaf(wg[w], mb_acc[(w * 8 + r) * SM::ACC_STRIDE + d], acc);
          p.part_acc[((size_t)my_slot * 8 + r) * D + d] = acc;
        }
        if (d0 == 0) { p.part_ml[my_slot * 16 + r] = mt; p.part_ml[my_slot * 16 + 8 + r] = lt; }
      }
    }

    if (!whole) {
      // ---- split unit: publish the partial; the CTA that arrives last combines ---------------------------------
      __threadfence();
      consumer_sync(NCONS);
      if (tid == 0) {
        const int old = atomicAdd(&p.tickets[unit_id], 1);
        const int last = (old == n_parts - 1) ? 1 : 0;
        if (last) p.tickets[unit_id] = 0;               // self-cleaning for the next launch
        misc[1] = last;
      }
      consumer_sync(NCONS);
      if (misc[1]) {
        __threadfence();
        // NCONS / 8 threads per query-head row, each with every TPR-th output dim.  The partials sit in L2: the loads
        // of two parts (their m, l and this thread's share of the accumulators) are issued together, so the combine
        // of a unit in two pieces costs two memory round trips -- it is the tail of the launch.
        constexpr int TPR = NCONS / 8;
        constexpr int PB = 2;                                   // parts whose loads are in flight together
        constexpr int DPT = (D + TPR - 1) / TPR;
        const int r = tid / TPR, d0 = tid - r * TPR;
        float mrun = -INFINITY, lrun = 0.f;
        float acc[DPT];
#pragma unroll
        for (int i = 0; i < DPT; ++i) acc[i] = 0.f;
        for (int c0 = 0; c0 < n_parts; c0 += PB) {
          float mw[PB], lw[PB], pa[PB][DPT];
#pragma unroll
          for (int u = 0; u < PB; ++u) {
            const int c = c0 + u;
            const bool okc = c < n_parts;
            const int slot = okc ? slot_base + c : slot_base;
            mw[u] = okc ? __ldcg(&p.part_ml[slot * 16 + r]) : -INFINITY;
            lw[u] = okc ? __ldcg(&p.part_ml[slot * 16 + 8 + r]) : 0.f;
#pragma unroll
            for (int i = 0; i < DPT; ++i) {
              const int d = d0 + i * TPR;
              pa[u][i] = (okc && d < D) ? __ldcg(&p.part_acc[((size_t)slot * 8 + r) * D + d]) : 0.f;
            }
          }
          float mnew = mrun;
#pragma unroll
          for (int u = 0; u < PB; ++u) mnew = fmaxf(mnew, mw[u]);
          if (c0 != 0) {                                        // more parts than one batch: rescale what is summed so far
            const float sc = (mrun == -INFINITY) ? 0.f : ex2(mrun - mnew);
            lrun *= sc;
#pragma unroll
            for (int i = 0; i < DPT; ++i) acc[i] *= sc;
          }
#pragma unroll
          for (int u = 0; u < PB; ++u) {
            const float wg = (mw[u] == -INFINITY) ? 0.f : ex2(mw[u] - mnew);
            lrun = fmaf(wg, lw[u], lrun);
#pragma unroll
            for (int i = 0; i < DPT; ++i) acc[i] = fmaf(wg, pa[u][i], acc[i]);
          }
          mrun = mnew;
        }
        if (r < g) {
#pragma unroll
          for (int i = 0; i < DPT; ++i) {
            const int d = d0 + i * TPR;
            if (d < D) out[(orow0 + r) * D + d] = __float2bfloat16_rn(acc[i] / lrun);
          }
          if (lse != nullptr && d0 == 0) lse[orow0 + r] = (mrun + log2f(lrun)) * 0.6931471805599453f;
          if (SCORE && d0 == 0)
            p.lse2[((size_t)(l0 + li) * B + b) * p.Hq + (size_t)h * g + r] = mrun + log2f(lrun);
        }
        if (SCORE && tid == 0) p.pending[(size_t)(l0 + li) * B + b] = 1;
      }
    }
    if (tid == 0) announce(useq + 1);
    consumer_sync(NCONS);       // merge buffers and misc[1] are free again; the verdict on the next item is posted
    ++useq;
  }
}

// ------------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn != nullptr) return fn;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(ptr);
  return fn;
}

bool make_ring_map(CUtensorMap* map, void* base, long long rows, int D, int tile_n) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)D * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)tile_n};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, PTENC_ATTN_L2PROMO,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int NW_DEFAULT = PTENC_ATTN_NW;
template <int D> struct Pick {
  static constexpr int TILE_N = (D == 128) ? PTENC_ATTN_TILE_N_128 : 64;
  static constexpr int STAGES = (D == 128) ? PTENC_ATTN_STAGES_128 : 12;
};
// Two instantiations per head size: four consumer warps (the default) and three.  With one lane issuing all tiles
// three warps used to sustain a little more bandwidth under the power cap on long launches; since every consumer warp
// has its own issuing lane four are as fast or faster at every shape measured (7B shape, 1500 back-to-back steps:
// 2.130 vs 2.147 ms; 512-token windows: 1.156 vs 1.220 ms), so the library no longer switches by itself.  The
// three-warp instantiation stays selectable through ptenc_config.attn_consumer_warps.
#ifndef PTENC_ATTN_NW_LONG
#define PTENC_ATTN_NW_LONG 3
#endif
constexpr int NW_LONG = PTENC_ATTN_NW_LONG;
inline bool use_long_variant(const ptenc_config& cfg, int nl, int tile_n) {
  (void)nl; (void)tile_n;
  return cfg.attn_consumer_warps == NW_LONG && NW_LONG != NW_DEFAULT;
}

// K and V tiles are read once per launch.  Marked "evict first", the tiles of a launch compete only with one another
// for L2, and what survives to the next step is a part of the rings instead of nothing: a call whose K/V bytes are a
// few times the 126 MB of L2 finds a part of them there.  Measured, hint on every launch against on none: 0.45 GiB of
// K/V per step -7.0 % step time, 0.89 GiB -3.3 %, 1.8 GiB -1.4 .. -3.6 %, 2.3 GiB (the 3B shape) -1.9 %, 3.5 GiB
// -0.4 %, 7 GiB +0.3 %, 14 GiB (the 7B shape) +2.1 %, 28 .. 56 GiB +1 .. 2 %: on the largest calls there is nothing to
// find and the hinted loads stream a little slower, so the hint is given up to 4 GiB only.
inline int ptenc_attn_kv_hint(int nl, const ptenc_config& cfg) {
  const unsigned long long bytes = 2ull * nl * cfg.batch * cfg.n_kv_heads * cfg.window * cfg.head_dim * 2ull;
  return bytes <= PTENC_ATTN_EVICT_FIRST_MAX_BYTES ? 1 : 0;
}

template <int D, int NW, bool SCORE>
cudaError_t launch_ts(ptenc_cache* c, int l0, int nl, const void* q, const uint8_t* active, void* out, float* lse,
                      bool fold_staged, bool early, cudaStream_t st) {
  constexpr int STAGES = Pick<D>::STAGES, TN = Pick<D>::TILE_N;
  using SM = Smem<D, TN, NW, STAGES>;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(c->attn_grid);
  cfg.blockDim = dim3((NW + 1 + PTENC_ATTN_ENC_WARPS) * 32);
  cfg.dynamicSmemBytes = SM::TOTAL + 1024;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (early) {
    // programmatic dependent launch: the grid may become resident and run its set-up while the kernel in front of it
    // on the stream (which signals that it allows this) is still running; the kernel waits before its first read
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  cudaError_t e = cudaLaunchKernelEx(&cfg, k_attn_bf16<D, TN, NW, STAGES, SCORE>, c->dev, c->tmK, c->tmV, l0, nl,
                                     (const __nv_bfloat16*)q, active, (__nv_bfloat16*)out, lse, fold_staged ? 1 : 0,
                                     ptenc_attn_kv_hint(nl, c->cfg));
  c->launches++;
  return e != cudaSuccess ? e : cudaGetLastError();
}
template <int D, int NW>
cudaError_t launch_t(ptenc_cache* c, int l0, int nl, const void* q, const uint8_t* active, void* out, float* lse,
                     bool fold_staged, bool early, cudaStream_t st) {
  return c->cfg.policy == PTENC_POLICY_SCORE
             ? launch_ts<D, NW, true>(c, l0, nl, q, active, out, lse, fold_staged, early, st)
             : launch_ts<D, NW, false>(c, l0, nl, q, active, out, lse, fold_staged, early, st);
}

template <int D, int NW>
cudaError_t prepare_nw() {
  constexpr int STAGES = Pick<D>::STAGES, TN = Pick<D>::TILE_N;
  using SM = Smem<D, TN, NW, STAGES>;
  cudaError_t e = cudaFuncSetAttribute(k_attn_bf16<D, TN, NW, STAGES, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL + 1024);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_attn_bf16<D, TN, NW, STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             SM::TOTAL + 1024);
  return e;
}
template <int D>
cudaError_t prepare_t() {
  cudaError_t e = prepare_nw<D, NW_DEFAULT>();
  if (e == cudaSuccess && NW_DEFAULT != NW_LONG) e = prepare_nw<D, NW_LONG>();
  return e;
}

}  // namespace

bool ptenc_attn_bf16_prepare(ptenc_cache* c, cudaError_t* err) {
  *err = cudaSuccess;
  const ptenc_config& cfg = c->cfg;
  if (cfg.dtype != PTENC_DTYPE_BF16) return false;
  if (cfg.head_dim != 128 && cfg.head_dim != 64) return false;
  if (c->dev.g > 8) return false;
  const long long rows = (long long)cfg.n_layers * cfg.batch * cfg.n_kv_heads * cfg.window;
  const int tile_n = cfg.head_dim == 128 ? Pick<128>::TILE_N : Pick<64>::TILE_N;
  if (!make_ring_map(&c->tmK, c->dev.K, rows, cfg.head_dim, tile_n)) return false;
  if (!make_ring_map(&c->tmV, c->dev.V, rows, cfg.head_dim, tile_n)) return false;
  *err = cfg.head_dim == 128 ? prepare_t<128>() : prepare_t<64>();
  if (*err != cudaSuccess) return false;
  c->attn_grid = c->sm_count * PTENC_ATTN_CTAS_PER_SM;
  if (2 * c->attn_grid > c->dev.part_slots) c->attn_grid = c->dev.part_slots / 2;
  return true;
}

void ptenc_attn_bf16_plan(const ptenc_cache* c, int nl, int* consumer_warps, int* tile_tokens, int* stages) {
  const bool d128 = c->cfg.head_dim == 128;
  const int tn = d128 ? Pick<128>::TILE_N : Pick<64>::TILE_N;
  *consumer_warps = use_long_variant(c->cfg, nl, tn) ? NW_LONG : NW_DEFAULT;
  *tile_tokens = tn;
  *stages = d128 ? Pick<128>::STAGES : Pick<64>::STAGES;
}

cudaError_t ptenc_launch_attn_bf16(ptenc_cache* c, int l0, int nl, const void* q, const uint8_t* active, void* out,
                                   float* lse, bool fold_staged, bool early, cudaStream_t st) {
  const bool d128 = c->cfg.head_dim == 128;
  const bool lng = use_long_variant(c->cfg, nl, d128 ? Pick<128>::TILE_N : Pick<64>::TILE_N);
  if (d128) return lng ? launch_t<128, NW_LONG>(c, l0, nl, q, active, out, lse, fold_staged, early, st)
                       : launch_t<128, NW_DEFAULT>(c, l0, nl, q, active, out, lse, fold_staged, early, st);
  return lng ? launch_t<64, NW_LONG>(c, l0, nl, q, active, out, lse, fold_staged, early, st)
             : launch_t<64, NW_DEFAULT>(c, l0, nl, q, active, out, lse, fold_staged, early, st);
}

// ================================================================================================================
// ptenc_attn_rings_static: the same attention kernel over KV rings the caller already owns, with the kernel's
// scratch (split partials, arrival tickets, status word) in a device array that is part of this library's image.
// Nothing is allocated: not by this code, not through the CUDA runtime, not through torch.
//
// For callers that cannot allocate device memory when they want to run attention: a serving process whose
// device memory was committed up front (rings, weights) and whose allocator is frozen, so a later cudaMalloc may
// fail or is forbidden by policy; a latency-critical loop that must not hit the device-wide synchronisation
// cudaMalloc / cudaFree imply.  Such a caller cannot build a ptenc workspace either, so this entry takes the rings
// and their head/count arrays directly.
// ================================================================================================================
namespace {

constexpr int STATIC_MAX_UNITS = 65536;                 // L * B * H_kv
constexpr int STATIC_MAX_SLOTS = 512;                   // two per CTA of the persistent grid
constexpr size_t STATIC_OFF_STATUS = 0;
constexpr size_t STATIC_OFF_TICKETS = 256;
constexpr size_t STATIC_OFF_ML = STATIC_OFF_TICKETS + (size_t)STATIC_MAX_UNITS * 4;
constexpr size_t STATIC_OFF_ACC = STATIC_OFF_ML + (size_t)STATIC_MAX_SLOTS * 16 * 4;
constexpr size_t STATIC_BYTES = STATIC_OFF_ACC + (size_t)STATIC_MAX_SLOTS * 8 * 128 * 4;   // 2,392,320 bytes

// Lives in every GPU that loads the library, from load to exit.  In host code this name is only a stand-in for
// the symbol, never a device address: the address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

constexpr int STATIC_MAX_DEVICES = 64;
struct StaticDevice {
  bool ready;
  unsigned char* scratch;     // device address of g_static_scratch on that device
  int sm_count;
};
StaticDevice g_static_dev[STATIC_MAX_DEVICES];

// Once per device, with that device current.
cudaError_t static_setup(int device, StaticDevice** out) {
  if (device < 0 || device >= STATIC_MAX_DEVICES) return cudaErrorInvalidDevice;
  StaticDevice& sd = g_static_dev[device];
  if (!sd.ready) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return e;
    e = prepare_t<128>();
    if (e != cudaSuccess) return e;
    e = prepare_t<64>();
    if (e != cudaSuccess) return e;
    sd.scratch = static_cast<unsigned char*>(ptr);
    sd.sm_count = sms;
    sd.ready = true;
  }
  *out = &sd;
  return cudaSuccess;
}

template <int D, int NW>
cudaError_t launch_static_t(const PtencDev& dev, const CUtensorMap& tmK, const CUtensorMap& tmV, int grid, int nl,
                            const void* q, const uint8_t* active, void* out, float* lse, int kv_hint, cudaStream_t st) {
  constexpr int STAGES = Pick<D>::STAGES, TN = Pick<D>::TILE_N;
  using SM = Smem<D, TN, NW, STAGES>;
  k_attn_bf16<D, TN, NW, STAGES, false><<<grid, (NW + 1 + PTENC_ATTN_ENC_WARPS) * 32, SM::TOTAL + 1024, st>>>(
      dev, tmK, tmV, 0, nl, (const __nv_bfloat16*)q, active, (__nv_bfloat16*)out, lse, 0, kv_hint);
  return cudaGetLastError();
}

}  // namespace

extern "C" int ptenc_attn_rings_static(const ptenc_config* cfg, const void* K, const void* V, const int32_t* head,
                                       const int32_t* count, const void* q, const uint8_t* active, void* out,
                                       float* lse_out, int32_t* status_out, void* stream) {
  if (cfg == nullptr || K == nullptr || V == nullptr || head == nullptr || count == nullptr || q == nullptr ||
      out == nullptr)
    return PTENC_EINVAL;
  if (cfg->n_layers <= 0 || cfg->batch <= 0 || cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0 || cfg->window <= 0 ||
      cfg->device < 0)
    return PTENC_EINVAL;
  if (cfg->attn_consumer_warps != 0 && cfg->attn_consumer_warps != 3 && cfg->attn_consumer_warps != 4)
    return PTENC_EINVAL;
  if (cfg->n_q_heads % cfg->n_kv_heads != 0) return PTENC_ESHAPE;
  if (cfg->dtype != PTENC_DTYPE_BF16 || (cfg->head_dim != 64 && cfg->head_dim != 128) ||
      cfg->n_q_heads / cfg->n_kv_heads > 8)
    return PTENC_ESHAPE;                      // only the tensor-core kernel uses scratch and has this variant
  const long long units = (long long)cfg->n_layers * cfg->batch * cfg->n_kv_heads;
  const long long rows = units * cfg->window;
  if (units > STATIC_MAX_UNITS || rows >= (1ll << 31)) return PTENC_ELIMIT;
  if (((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) | reinterpret_cast<uintptr_t>(q) |
        reinterpret_cast<uintptr_t>(out)) & 15) != 0)
    return PTENC_EALIGN;

  // Like every other entry point this one leaves the caller's current device alone: cfg->device has to be current.
  int cur_dev = -1;
  if (cudaGetDevice(&cur_dev) != cudaSuccess) return PTENC_ECUDA;
  if (cur_dev != cfg->device) return PTENC_EINVAL;
  StaticDevice* sd = nullptr;
  if (static_setup(cfg->device, &sd) != cudaSuccess) return PTENC_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  CUtensorMap tmK, tmV;
  const int tile_n = cfg->head_dim == 128 ? Pick<128>::TILE_N : Pick<64>::TILE_N;
  if (!make_ring_map(&tmK, const_cast<void*>(K), rows, cfg->head_dim, tile_n)) return PTENC_ECUDA;
  if (!make_ring_map(&tmV, const_cast<void*>(V), rows, cfg->head_dim, tile_n)) return PTENC_ECUDA;

  PtencDev d;
  memset(&d, 0, sizeof(d));
  d.L = cfg->n_layers; d.B = cfg->batch; d.Hq = cfg->n_q_heads; d.Hkv = cfg->n_kv_heads; d.D = cfg->head_dim;
  d.W = cfg->window; d.g = d.Hq / d.Hkv; d.d_q = d.Hq * d.D; d.d_kv = d.Hkv * d.D;
  d.dtype = PTENC_DTYPE_BF16; d.elt = 2;
  d.K = static_cast<char*>(const_cast<void*>(K));
  d.V = static_cast<char*>(const_cast<void*>(V));
  d.head = const_cast<int*>(head);
  d.count = const_cast<int*>(count);
  d.status = reinterpret_cast<int*>(sd->scratch + STATIC_OFF_STATUS);
  d.work = reinterpret_cast<int*>(sd->scratch + STATIC_OFF_STATUS + 16);
  d.tickets = reinterpret_cast<int*>(sd->scratch + STATIC_OFF_TICKETS);
  d.part_ml = reinterpret_cast<float*>(sd->scratch + STATIC_OFF_ML);
  d.part_acc = reinterpret_cast<float*>(sd->scratch + STATIC_OFF_ACC);
  d.part_slots = STATIC_MAX_SLOTS;
  int grid = sd->sm_count * PTENC_ATTN_CTAS_PER_SM;
  if (2 * grid > STATIC_MAX_SLOTS) grid = STATIC_MAX_SLOTS / 2;
  const int kv_hint = ptenc_attn_kv_hint(cfg->n_layers, *cfg);

  // The array keeps whatever the last call left: the status word, the work counter and the tickets must start at zero.
  if (cudaMemsetAsync(sd->scratch, 0, STATIC_OFF_TICKETS + (size_t)units * 4, st) != cudaSuccess) return PTENC_ECUDA;
  // the same choice of instantiation as ptenc_decode_attn makes for a call over all layers
  const bool lng = use_long_variant(*cfg, cfg->n_layers, tile_n);
  cudaError_t e;
  if (cfg->head_dim == 128)
    e = lng ? launch_static_t<128, NW_LONG>(d, tmK, tmV, grid, cfg->n_layers, q, active, out, lse_out, kv_hint, st)
            : launch_static_t<128, NW_DEFAULT>(d, tmK, tmV, grid, cfg->n_layers, q, active, out, lse_out, kv_hint, st);
  else
    e = lng ? launch_static_t<64, NW_LONG>(d, tmK, tmV, grid, cfg->n_layers, q, active, out, lse_out, kv_hint, st)
            : launch_static_t<64, NW_DEFAULT>(d, tmK, tmV, grid, cfg->n_layers, q, active, out, lse_out, kv_hint, st);
  if (e != cudaSuccess) return PTENC_ECUDA;
  if (status_out != nullptr &&
      cudaMemcpyAsync(status_out, d.status, 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return PTENC_ECUDA;
  return PTENC_OK;
}
