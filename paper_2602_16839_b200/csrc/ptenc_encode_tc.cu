// Progressive encoder (step a3) for a chunk of evicted tokens, on the sm_100a tensor cores.
//
// Sec. 3.3, Eq. (3): S' = ((W^a_Q q_g)(W^a_K K_e)^T)(W^a_V V_e), S <- Normalize(S + S').  Sec. 4.1: when the cache
// saturates a fraction of it (a chunk of E tokens, 25 % in the paper's runs) is evicted at once, so K_e, V_e are
// [m, d_kv] with m in the hundreds and the two projections K_a = K_e W^a_K^T, V_a = V_e W^a_V^T are dense
// contractions over d_kv (~ r flop per byte read): the one place on this path where the tensor cores are needed
// to stay on the HBM roofline.
//
// CTAs (two per SM) walk the (layer, sequence) units that have evicted rows; per CTA:
//  * warp 0 (one lane): TMA producer.  Per pipeline item it loads a [rows x 64] slab of the evicted K (or V) rows
//    and the matching [r x 64] slab of W^a_K (or W^a_V), both K-major with the 128-byte swizzle, into a stage
//    guarded by full/empty mbarriers.  Plain per-CTA loads of this GPU's own memory.
//  * warp 1 (one lane): issues tcgen05.mma (M = 128 token rows, N = r, K = 16, bf16 x bf16 -> fp32) with the
//    accumulators in tensor memory: K_a in columns [0, r), V_a in [r, 2r) of one of two buffers, so the epilogue
//    of a 128-token tile overlaps the loads and MMAs of the next one.  tcgen05.commit releases the stages and
//    publishes the tile.
//  * warps 2..5: epilogue.  Each thread owns one token row (one TMEM lane): tcgen05.ld its k_a and v_a, zero the
//    rows past the chunk, and accumulate M2 += K_a^T V_a [r, r] in fp32 through shared memory.  After the last
//    tile S' = Q_a M2 (the bracketed product re-associated: (Q_a K_a^T) V_a = Q_a (K_a^T V_a)), S + S', Normalize.
//  Everything after the projections is fp32 FMA: rounding k_a, v_a to bf16 for a second tensor-core pass would
//  cost three decimal digits of the state.
//  * Every mbarrier wait is bounded; a wait that runs out sets a status bit and an abort flag, every role then
//    leaves its loop, copies and MMAs in flight are drained with bounded waits, and tensor memory is freed.
#include <string.h>

#include "ptenc_internal.h"

namespace {

constexpr uint32_t TC_WAIT_POLLS = 4000000;
constexpr int TC_M = 128;            // token rows per MMA tile = TMEM lanes
constexpr int TC_KC = 64;            // contraction values per pipeline item: one 128-byte swizzled row of bf16
constexpr int TC_STAGES = 3;
constexpr int TC_THREADS = 192;      // warp 0 producer, warp 1 MMA + TMEM owner, warps 2..5 epilogue
constexpr int TC_EPI = 128;

// ------------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t tc_smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void tc_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void tc_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t tc_mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait that also gives up when another role has raised the abort flag.
__device__ __forceinline__ bool tc_mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < TC_WAIT_POLLS; ++i) {
    if (tc_mbar_test(bar, parity)) return true;
    if (i > 64) __nanosleep(64);
    if ((i & 255) == 255 && *abort_flag != 0) return false;
  }
  return false;
}
__device__ __forceinline__ void tc_tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], M = 128, N and dtypes in idesc; one thread issues.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier gets one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void tc_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tc_cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void tc_epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(TC_EPI) : "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile stored with the 128-byte swizzle (rows of 128 bytes,
// groups of 8 rows 1024 bytes apart, tile base 1024-byte aligned).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused with a swizzled K-major tile)
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset: next group of 8 rows
  d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                            // layout: 128-byte swizzle
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t tc_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TC_M >> 4) << 24);
}

template <int R>
struct TcSmem {
  static constexpr int A_BYTES = TC_M * TC_KC * 2;                  // 16 KiB (a_rows <= 128 of them are loaded)
  static constexpr int W_BYTES = R * TC_KC * 2;
  static constexpr int STAGE_BYTES = A_BYTES + W_BYTES;
  static constexpr int RP = R + 4;                                  // row pitch of k_a / v_a: 16-byte stores of
                                                                    // consecutive rows fall into distinct banks
  static constexpr int OFF_KA = TC_STAGES * STAGE_BYTES;            // fp32 [128][RP]
  static constexpr int OFF_VA = OFF_KA + TC_M * RP * 4;             // fp32 [128][RP], directly behind k_a
  static constexpr int OFF_M2 = OFF_VA + TC_M * RP * 4;             // fp32 [R][R]
  static constexpr int OFF_BAR = OFF_M2 + R * R * 4;                // mbarriers, TMEM base, flags
  static constexpr int OFF_QA = OFF_BAR + 128;                      // fp32 [G][R] Q_a, then [G][R] old state rows
  static size_t total(int G) { return (size_t)OFF_QA + (size_t)2 * G * R * 4 + 1024; }
  static_assert(OFF_VA % 16 == 0 && OFF_M2 % 16 == 0 && STAGE_BYTES % 1024 == 0 && W_BYTES % 1024 == 0, "alignment");
  static_assert(2 * TC_M * RP * 4 >= TC_M * 32 * 4, "the groups' partial sums fit over the row buffers");
};

struct TcArgs {
  int l0;             // first layer of the call
  int a_rows;         // rows of the A box (multiple of 8, <= 128)
  int rows_per_seq;   // row pitch between sequences in the A tensors (E for the staged rows, m_max for caller rows)
  int staged;         // 1: m comes from n_staged and layers are absolute; 0: from n_ev, layers relative to l0
  const int32_t* n_ev;
  int m_max;
  int nl;             // layers of the call
};

template <int R>
__global__ void __launch_bounds__(TC_THREADS)
k_encode_chunk_tc(const PtencDev p, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const __grid_constant__ CUtensorMap tmWk, const __grid_constant__ CUtensorMap tmWv,
                  const TcArgs a) {
  using SM = TcSmem<R>;
  constexpr uint32_t TMEM_COLS = (4 * R < 32) ? 32 : 4 * R;         // two buffers of (k_a | v_a); power of two
  static_assert(R == 16 || R == 32 || R == 64, "rank");

  extern __shared__ uint8_t tc_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = tc_smem_u32(smem);
  float* ka_s = reinterpret_cast<float*>(smem + SM::OFF_KA);
  float* va_s = reinterpret_cast<float*>(smem + SM::OFF_VA);
  float* m2_s = reinterpret_cast<float*>(smem + SM::OFF_M2);
  float* qa_s = reinterpret_cast<float*>(smem + SM::OFF_QA);
  float* so_s = qa_s + (size_t)p.G * R;
  const uint32_t bar_full = sbase + SM::OFF_BAR;                     // [TC_STAGES]
  const uint32_t bar_empty = bar_full + 8 * TC_STAGES;               // [TC_STAGES]
  const uint32_t bar_tfull = bar_empty + 8 * TC_STAGES;              // [2]
  const uint32_t bar_tempty = bar_tfull + 16;                        // [2]
  const uint32_t bar_drain = bar_tempty + 16;                        // [1]
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + SM::OFF_BAR + 8 * (2 * TC_STAGES + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* frob = reinterpret_cast<float*>(const_cast<uint32_t*>(tmem_slot) + 2);   // [4]
  volatile int* epi_abort = reinterpret_cast<volatile int*>(tmem_slot + 6);      // written by epilogue threads only

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int B = p.B, G = p.G, d_kv = p.d_kv;
  if (!p.encode_enabled) return;
  const int n_units = a.nl * B;
  const int nkc = d_kv / TC_KC;
  const uint32_t tx_bytes = (uint32_t)(a.a_rows * TC_KC * 2 + SM::W_BYTES);
  // The CTA walks the (layer, sequence) units u = blockIdx.x, blockIdx.x + gridDim.x, ...; every role takes the same
  // walk and skips the same units (no encoder for the layer, nothing evicted).  Returns the unit's row count.
  auto unit = [&](int u, int* l, int* b, long long* row0) -> int {
    const int li = u / B;
    *b = u - li * B;
    *l = a.l0 + li;
    if (!p.enc_set[*l]) return 0;
    int m;
    if (a.staged) {
      m = p.n_staged[(size_t)(*l) * B + *b];
      *row0 = ((long long)(*l) * B + *b) * a.rows_per_seq;
    } else {
      m = a.n_ev[(size_t)li * B + *b];
      if (m > a.m_max) m = a.m_max;
      *row0 = ((long long)li * B + *b) * a.rows_per_seq;
    }
    return m > 0 ? m : 0;
  };

  // Most steps of a chunked rollout evict nothing: look at this CTA's units first and leave before any set-up.
  {
    int any = 0;
    for (int u = blockIdx.x + tid * gridDim.x; u < n_units; u += TC_THREADS * gridDim.x) {
      int l, b;
      long long row0;
      any |= unit(u, &l, &b, &row0) > 0 ? 1 : 0;
    }
    if (__syncthreads_or(any) == 0) return;
  }

  if (tid == 0) {
    for (int s = 0; s < TC_STAGES; ++s) { tc_mbar_init(bar_full + 8 * s, 1); tc_mbar_init(bar_empty + 8 * s, 1); }
    for (int i = 0; i < 2; ++i) { tc_mbar_init(bar_tfull + 8 * i, 1); tc_mbar_init(bar_tempty + 8 * i, 4); }
    tc_mbar_init(bar_drain, 1);
    *abort_flag = 0;
    *epi_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // A rows that the box does not cover are never written by TMA: clear the stages once so that the MMA reads finite
  // values there (those token rows are discarded anyway, but keep them tame).
  if (a.a_rows < TC_M)
    for (int i = tid; i < TC_STAGES * SM::STAGE_BYTES / 16; i += TC_THREADS)
      reinterpret_cast<uint4*>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    tc_tmem_alloc(tc_smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
    tc_tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ================================================================ producer
    if (lane == 0) {
      uint32_t n = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        int l, b;
        long long row0;
        const int m = unit(u, &l, &b, &row0);
        const int n_tiles = (m + a.a_rows - 1) / a.a_rows;
        for (int tile = 0; tile < n_tiles && ok; ++tile) {
          const int y = (int)(row0 + (long long)tile * a.a_rows);
          for (int mat = 0; mat < 2 && ok; ++mat) {
            for (int kc = 0; kc < nkc; ++kc, ++n) {
              const uint32_t s = n % TC_STAGES;
              if (!tc_mbar_wait(bar_empty + 8 * s, ((n / TC_STAGES) & 1) ^ 1, abort_flag)) { ok = false; break; }
              const uint32_t dst = sbase + s * SM::STAGE_BYTES;
              const uint32_t fb = bar_full + 8 * s;
              tc_mbar_expect_tx(fb, tx_bytes);
              tc_tma_load_2d(dst, mat ? &tmV : &tmK, kc * TC_KC, y, fb);
              tc_tma_load_2d(dst + SM::A_BYTES, mat ? &tmWv : &tmWk, kc * TC_KC, l * R, fb);
            }
          }
        }
      }
      if (!ok) {
        atomicOr(p.status, PTENC_ST_WAIT_TIMEOUT);
        *abort_flag = 1;
        // copies in flight must land before this CTA's shared memory is released
        const uint32_t back = n < (uint32_t)TC_STAGES ? n : (uint32_t)TC_STAGES;
        for (uint32_t i = 0; i < back; ++i) {
          const uint32_t nn = n - 1 - i;
          for (uint32_t k = 0; k < TC_WAIT_POLLS; ++k)
            if (tc_mbar_test(bar_full + 8 * (nn % TC_STAGES), (nn / TC_STAGES) & 1)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC = tc_idesc(R);
      uint32_t n = 0, gt = 0;                           // pipeline items and 128-token tiles issued so far
      bool ok = true;
      for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        int l, b;
        long long row0;
        const int m = unit(u, &l, &b, &row0);
        const int n_tiles = (m + a.a_rows - 1) / a.a_rows;
        for (int tile = 0; tile < n_tiles && ok; ++tile, ++gt) {
          const uint32_t bf = gt & 1;
          if (!tc_mbar_wait(bar_tempty + 8 * bf, ((gt >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          for (int mat = 0; mat < 2 && ok; ++mat) {
            const uint32_t d_tmem = tmem_base + bf * 2 * R + mat * R;
            for (int kc = 0; kc < nkc; ++kc, ++n) {
              const uint32_t s = n % TC_STAGES;
              if (!tc_mbar_wait(bar_full + 8 * s, (n / TC_STAGES) & 1, abort_flag)) { ok = false; break; }
              tc_fence_after();
              const uint32_t a_addr = sbase + s * SM::STAGE_BYTES;
              const uint32_t w_addr = a_addr + SM::A_BYTES;
#pragma unroll
              for (int k4 = 0; k4 < TC_KC / 16; ++k4)
                tc_mma(d_tmem, tc_smem_desc(a_addr + 32 * k4), tc_smem_desc(w_addr + 32 * k4), IDESC,
                       (kc > 0 || k4 > 0) ? 1u : 0u);
              tc_commit(bar_empty + 8 * s);
            }
          }
          if (ok) tc_commit(bar_tfull + 8 * bf);
        }
      }
      if (!ok) {
        atomicOr(p.status, PTENC_ST_WAIT_TIMEOUT);
        *abort_flag = 1;
        tc_commit(bar_drain);                          // MMAs still in flight finish before TMEM is freed
        for (uint32_t k = 0; k < TC_WAIT_POLLS; ++k)
          if (tc_mbar_test(bar_drain, 0)) break;
      }
    }
  } else {
    // ================================================================ epilogue: 128 threads, one token row each
    // M2 += K_a^T V_a runs on 4 x 8 register blocks: SLOTS threads cover the r x r result once, and the 128 threads
    // form COPIES such groups that each sum the token rows of their own (for r <= 32 a group lies inside one warp
    // and sums rows that this warp wrote, so a warp barrier orders the exchange).  Every shared-memory value then
    // feeds four or eight FMAs; one value per FMA made shared-memory bandwidth the bound of the whole kernel.
    constexpr int RP = SM::RP;
    constexpr int SLOTS = R * R / 32;
    constexpr int COPIES = TC_EPI / SLOTS;              // 16, 4, 1 for r = 16, 32, 64
    constexpr int KG = R / 8;
    constexpr bool WARP_LOCAL = COPIES >= 4;
    const int et = tid - 64;                            // 0..127
    const int q = warp & 3;                             // TMEM lane quarter this warp may read
    const int row = 32 * q + lane;
    const int ew = et >> 5;
    const int slot = et % SLOTS, copy = et / SLOTS;
    const int j0 = (slot / KG) * 4, k0 = (slot % KG) * 8;
    const int rr0 = WARP_LOCAL ? 32 * q + (lane / SLOTS) * SLOTS : 0;
    float* part = ka_s;                                 // [COPIES][R][R], over the row buffers once they are idle
    uint32_t gt = 0;                                    // 128-token tiles consumed so far
    bool ok = true;
    int l = 0, b = 0, m = 0;
    long long row0 = 0;
    int u = blockIdx.x;
    if (u < n_units) m = unit(u, &l, &b, &row0);
    while (u < n_units && ok) {
      // the next unit's description is requested now and used after this unit
      const int u_next = u + (int)gridDim.x;
      int l_next = 0, b_next = 0, m_next = 0;
      long long row0_next = 0;
      if (u_next < n_units) m_next = unit(u_next, &l_next, &b_next, &row0_next);
      if (m > 0) {                                       // uniform over the CTA
        const int n_tiles = (m + a.a_rows - 1) / a.a_rows;
        float* S = p.S + ((size_t)l * B + b) * G * R;
        // Q_a of the unit's layer and the old state rows travel to shared memory while the tiles are reduced (the
        // previous unit's last reads of these buffers are behind this barrier)
        tc_epi_sync();
        for (int i = et; i < G * R / 4; i += TC_EPI) {
          tc_cp_async16(tc_smem_u32(qa_s + 4 * i), p.Qa + (size_t)l * G * R + 4 * i);
          tc_cp_async16(tc_smem_u32(so_s + 4 * i), S + 4 * i);
        }
        tc_cp_async_commit();
        float acc[4][8];
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
          for (int y = 0; y < 8; ++y) acc[x][y] = 0.f;
        for (int tile = 0; tile < n_tiles && ok; ++tile, ++gt) {
          const uint32_t bf = gt & 1;
          // The four warps must agree on going on: the barriers below count all 128 threads.  Each thread reports
          // its own wait, thread 0 adds the other roles' flag, and everybody reads the verdict after a barrier
          // (which also orders the previous tile's reads of the row buffers before this tile's writes).
          if (!tc_mbar_wait(bar_tfull + 8 * bf, (gt >> 1) & 1, abort_flag)) *epi_abort = 1;
          if (et == 0 && *abort_flag != 0) *epi_abort = 1;
          tc_epi_sync();
          if (*epi_abort != 0) { ok = false; break; }
          tc_fence_after();
          {
            float kr[R], vr[R];
            const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + bf * 2 * R;
#pragma unroll
            for (int c = 0; c < R; c += 16) {
              tc_ld16(taddr + c, kr + c);
              tc_ld16(taddr + R + c, vr + c);
            }
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(bar_tempty + 8 * bf);
            const bool valid = (row < a.a_rows) && (tile * a.a_rows + row < m);
            const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < R; j += 4) {
              *reinterpret_cast<float4*>(ka_s + row * RP + j) =
                  valid ? make_float4(kr[j], kr[j + 1], kr[j + 2], kr[j + 3]) : zero;
              *reinterpret_cast<float4*>(va_s + row * RP + j) =
                  valid ? make_float4(vr[j], vr[j + 1], vr[j + 2], vr[j + 3]) : zero;
            }
          }
          if (WARP_LOCAL) __syncwarp(); else tc_epi_sync();
          // acc[x][y] += sum over this group's rows of k_a[row][j0 + x] * v_a[row][k0 + y]
#pragma unroll 4
          for (int rr = rr0; rr < rr0 + SLOTS; ++rr) {
            const float4 k4 = *reinterpret_cast<const float4*>(ka_s + rr * RP + j0);
            const float4 va = *reinterpret_cast<const float4*>(va_s + rr * RP + k0);
            const float4 vb = *reinterpret_cast<const float4*>(va_s + rr * RP + k0 + 4);
            const float kx[4] = {k4.x, k4.y, k4.z, k4.w};
            const float vy[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
              for (int y = 0; y < 8; ++y) acc[x][y] = fmaf(kx[x], vy[y], acc[x][y]);
          }
        }
        if (!ok) break;                                 // uniform: the verdict was read after a barrier
        // the groups' sums meet in shared memory
        if (COPIES > 1) {
          tc_epi_sync();                                // every group is done with the row buffers
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            float* dst = part + (size_t)copy * R * R + (j0 + x) * R + k0;
            *reinterpret_cast<float4*>(dst) = make_float4(acc[x][0], acc[x][1], acc[x][2], acc[x][3]);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[x][4], acc[x][5], acc[x][6], acc[x][7]);
          }
          tc_epi_sync();
          for (int o = et; o < R * R / 4; o += TC_EPI) {
            float4 t = *reinterpret_cast<const float4*>(part + 4 * o);
#pragma unroll
            for (int c = 1; c < COPIES; ++c) {
              const float4 w = *reinterpret_cast<const float4*>(part + (size_t)c * R * R + 4 * o);
              t.x += w.x; t.y += w.y; t.z += w.z; t.w += w.w;
            }
            *reinterpret_cast<float4*>(m2_s + 4 * o) = t;
          }
        } else {
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            float* dst = m2_s + (j0 + x) * R + k0;
            *reinterpret_cast<float4*>(dst) = make_float4(acc[x][0], acc[x][1], acc[x][2], acc[x][3]);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[x][4], acc[x][5], acc[x][6], acc[x][7]);
          }
        }
        tc_cp_async_wait_all();
        tc_epi_sync();                                  // M2, Q_a and the old state rows are in shared memory
        // S' = Q_a M2, S <- Normalize(S + S'): epilogue warp w takes state rows w, w + 4, ..., eight at a time, a
        // lane per column
        constexpr int JJ = (R + 31) / 32;
        constexpr int ROWS = 8;
        float total = 0.f;
        for (int g0 = 0; g0 < G; g0 += 4 * ROWS) {
          float sp[ROWS][JJ];
#pragma unroll
          for (int i = 0; i < ROWS; ++i)
#pragma unroll
            for (int jj = 0; jj < JJ; ++jj) sp[i][jj] = 0.f;
#pragma unroll 2
          for (int j = 0; j < R; j += 4) {
            float mm[4][JJ];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
              for (int jj = 0; jj < JJ; ++jj) {
                const int k = lane + 32 * jj;
                mm[t][jj] = (k < R) ? m2_s[(j + t) * R + k] : 0.f;
              }
#pragma unroll
            for (int i = 0; i < ROWS; ++i) {
              const int gi = min(g0 + ew + 4 * i, G - 1);          // rows past G are computed and dropped
              const float4 q4 = *reinterpret_cast<const float4*>(qa_s + gi * R + j);
#pragma unroll
              for (int jj = 0; jj < JJ; ++jj)
                sp[i][jj] = fmaf(q4.x, mm[0][jj], fmaf(q4.y, mm[1][jj], fmaf(q4.z, mm[2][jj], fmaf(q4.w, mm[3][jj], sp[i][jj]))));
            }
          }
          // the eight rows' sums of squares are reduced side by side (eight shuffles in flight, not a chain of forty)
          float val[ROWS][JJ], ss[ROWS];
#pragma unroll
          for (int i = 0; i < ROWS; ++i) {
            const int gi = min(g0 + ew + 4 * i, G - 1);
            ss[i] = 0.f;
#pragma unroll
            for (int jj = 0; jj < JJ; ++jj) {
              const int k = lane + 32 * jj;
              val[i][jj] = (k < R) ? so_s[gi * R + k] + sp[i][jj] : 0.f;
              ss[i] = fmaf(val[i][jj], val[i][jj], ss[i]);
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int i = 0; i < ROWS; ++i) ss[i] += __shfl_xor_sync(0xffffffffu, ss[i], o);
#pragma unroll
          for (int i = 0; i < ROWS; ++i) {
            const int gi = g0 + ew + 4 * i;
            if (gi < G) {                                   // uniform over the warp
              total += ss[i];
              const float sc = (p.norm_mode == PTENC_NORM_ROW_L2) ? 1.f / fmaxf(sqrtf(ss[i]), 1e-12f) : 1.f;
#pragma unroll
              for (int jj = 0; jj < JJ; ++jj) {
                const int k = lane + 32 * jj;
                if (k < R) S[gi * R + k] = val[i][jj] * sc;
              }
            }
          }
        }
        if (p.norm_mode == PTENC_NORM_FROBENIUS) {
          if (lane == 0) frob[ew] = total;
          tc_epi_sync();
          const float sc = 1.f / fmaxf(sqrtf(frob[0] + frob[1] + frob[2] + frob[3]), 1e-12f);
          for (int gi = ew; gi < G; gi += 4)
            for (int k = lane; k < R; k += 32) S[gi * R + k] *= sc;      // each lane rescales what it stored
        }
      }
      u = u_next; l = l_next; b = b_next; m = m_next; row0 = row0_next;
    }
    // after an abort the remaining units are left untouched
    if (!ok && lane == 0) { atomicOr(p.status, PTENC_ST_WAIT_TIMEOUT); *abort_flag = 1; }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tc_tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------ host
typedef CUresult (*TcEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

TcEncodeTiledFn tc_encode_fn() {
  static TcEncodeTiledFn fn = nullptr;
  if (fn != nullptr) return fn;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<TcEncodeTiledFn>(ptr);
  return fn;
}

// 2-D bf16 tensor [rows][cols], box [box_rows][64], 128-byte swizzle.
bool tc_make_map(CUtensorMap* map, const void* base, long long rows, int cols, int box_rows) {
  TcEncodeTiledFn fn = tc_encode_fn();
  if (fn == nullptr || rows <= 0) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)TC_KC, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int tc_box_rows(int rows_per_seq) {
  int r8 = (rows_per_seq + 7) / 8 * 8;
  return r8 < TC_M ? r8 : TC_M;
}

template <int R>
cudaError_t tc_launch(ptenc_cache* c, const CUtensorMap& tmK, const CUtensorMap& tmV, const TcArgs& a, int nl,
                      cudaStream_t st) {
  const size_t smem = TcSmem<R>::total(c->dev.G);
  static bool attr_done[PTENC_MAX_DEVICES] = {};
  if (ptenc_first_use(attr_done, c->cfg.device)) {
    cudaError_t e = cudaFuncSetAttribute(k_encode_chunk_tc<R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)TcSmem<R>::total(128));
    if (e != cudaSuccess) return e;
  }
  // persistent: two CTAs per SM walk the (layer, sequence) units, so barriers and tensor memory are set up once per
  // CTA and the loads of a unit's first tile overlap the epilogue of the unit before
  int grid = nl * c->cfg.batch;
  if (grid > 2 * c->sm_count) grid = 2 * c->sm_count;
  k_encode_chunk_tc<R><<<grid, TC_THREADS, smem, st>>>(c->dev, tmK, tmV, c->tmWk, c->tmWv, a);
  c->launches++;
  return cudaGetLastError();
}

}  // namespace

// Shapes the tensor-core chunk encoder covers: bf16 storage, rank 16/32/64, d_kv a multiple of 64.
bool ptenc_encode_tc_prepare(ptenc_cache* c) {
  c->tc_encode = false;
  const PtencDev& p = c->dev;
  if (c->cfg.dtype != PTENC_DTYPE_BF16) return false;
  if (p.r != 16 && p.r != 32 && p.r != 64) return false;
  if ((p.d_kv % TC_KC) != 0) return false;
  if (!tc_make_map(&c->tmWk, p.Wk, (long long)p.L * p.r, p.d_kv, p.r)) return false;
  if (!tc_make_map(&c->tmWv, p.Wv, (long long)p.L * p.r, p.d_kv, p.r)) return false;
  const long long rows = (long long)p.L * p.B * p.E;
  if (rows >= (1ll << 31)) return false;
  c->tc_stage_box = tc_box_rows(p.E);
  if (rows < c->tc_stage_box) return false;
  if (!tc_make_map(&c->tmStageK, p.stageK, rows, p.d_kv, c->tc_stage_box)) return false;
  if (!tc_make_map(&c->tmStageV, p.stageV, rows, p.d_kv, c->tc_stage_box)) return false;
  c->tc_encode = true;
  return true;
}

// Ke == nullptr: the rows staged by the last append.  Otherwise caller rows [nl][B][m_max][d_kv].
cudaError_t ptenc_launch_encode_tc(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve,
                                   const int32_t* n_ev, int m_max, cudaStream_t st) {
  const PtencDev& p = c->dev;
  TcArgs a;
  memset(&a, 0, sizeof(a));
  a.l0 = l0;
  a.nl = nl;
  CUtensorMap tmK, tmV;
  if (Ke == nullptr) {
    a.staged = 1;
    a.rows_per_seq = p.E;
    a.a_rows = c->tc_stage_box;
    tmK = c->tmStageK;
    tmV = c->tmStageV;
  } else {
    a.staged = 0;
    a.rows_per_seq = m_max;
    a.a_rows = tc_box_rows(m_max);
    a.n_ev = n_ev;
    a.m_max = m_max;
    const long long rows = (long long)nl * p.B * m_max;
    if (rows >= (1ll << 31)) return cudaErrorInvalidValue;
    if (!tc_make_map(&tmK, Ke, rows, p.d_kv, a.a_rows) || !tc_make_map(&tmV, Ve, rows, p.d_kv, a.a_rows))
      return cudaErrorInvalidValue;
  }
  switch (p.r) {
    case 16: return tc_launch<16>(c, tmK, tmV, a, nl, st);
    case 32: return tc_launch<32>(c, tmK, tmV, a, nl, st);
    case 64: return tc_launch<64>(c, tmK, tmV, a, nl, st);
    default: return cudaErrorInvalidValue;
  }
}
