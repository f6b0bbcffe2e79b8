// Ring-per-step mode (E = 1): every arriving token evicts exactly one token once the ring is full, so steps a1 and
// a3 of a decode step touch one row per sequence.  This kernel does both for a block of 16 sequences of one layer:
//
//   a1 (Sec. 3.2 / 3.3, sliding-window policy): evict the oldest token when the ring is full -- its row is staged
//      and also kept in shared memory -- then write the arriving token into the freed slot and advance the ring.
//   a3 (Sec. 3.3, Eq. (3)): k_a = W^a_K k_e, v_a = W^a_V v_e, S' = (Q_a k_a) v_a^T, S <- Normalize(S + S').
//
// The 16 evicted rows form one small matrix product X [16, d_kv] x W^T [d_kv, r] per map, done with warp-level
// bf16 mma (fp32 accumulate), so a layer's weights are read once per 16 sequences instead of once per sequence.
// Each lane fetches 8 consecutive k-values of its A row (shared memory) and of its B row (W^a, from L2) with one
// 16-byte load and feeds them to two mma steps; the contraction index is permuted the same way on both operands,
// which leaves the sum unchanged.  The kernel is a chain of dependent memory round trips, so everything it will
// need later (its slice of the weights, Q_a, the sequences' state rows) is pulled into L2 with prefetches at the very
// start, while the ring state and the evicted rows are still on their way; two CTAs fit on an SM so that the whole
// grid of a 28-layer x 128-sequence step is resident at once.  Everything after the projections is fp32.
//
// The same kernel serves ptenc_encode alone (APPEND = false: rows come from the staging area or from the caller).
#include "ptenc_internal.h"

namespace {

constexpr int E1_SEQ = 16;                 // sequences per CTA = rows of the mma tile
constexpr int E1_THREADS = 512;
constexpr int E1_WARPS = E1_THREADS / 32;  // one warp per sequence in the row-wise phases

__device__ __forceinline__ void e1_prefetch_l2(const void* ptr) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}

__device__ __forceinline__ void e1_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                       uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct E1Args {
  int l0;
  const __nv_bfloat16* k_new;      // APPEND: [nl][B][Hkv][D]
  const __nv_bfloat16* v_new;
  const uint8_t* active;           // APPEND: [B] or null
  const __nv_bfloat16* Ke;         // !APPEND: caller rows [nl][B][1][d_kv] or null = staged rows
  const __nv_bfloat16* Ve;
  const int32_t* n_ev;
  int k_split;                     // warps that share one column tile of the projections
};

__host__ __device__ inline int e1_k_split(int r) {
  const int tiles = 2 * (r >> 3);
  int ks = E1_WARPS / tiles;
  return ks < 1 ? 1 : ks;
}

__host__ __device__ inline size_t e1_smem_bytes(int G, int r, int d_kv) {
  const size_t xstride = (size_t)d_kv * 2 + 64;
  return 2 * E1_SEQ * xstride +
         sizeof(float) * ((size_t)e1_k_split(r) * E1_SEQ * 2 * r + (size_t)G * (r + 1) + (size_t)E1_SEQ * G) +
         E1_SEQ * sizeof(int);
}

// RJ = ceil(r / 32): state elements of one row held by a lane.
template <bool APPEND, int RJ>
__global__ void __launch_bounds__(E1_THREADS, 2)
k_step_e1(PtencDev p, E1Args a) {
  extern __shared__ __align__(16) uint8_t e1_smem[];
  const int G = p.G, r = p.r, d_kv = p.d_kv, B = p.B, W = p.W;
  const int xstride = d_kv * 2 + 64;                 // bytes; = 64 mod 128 keeps the 16-byte A loads conflict-free
  const int KS = a.k_split;
  uint8_t* xk = e1_smem;
  uint8_t* xv = xk + E1_SEQ * xstride;
  float* kv_a = reinterpret_cast<float*>(xv + E1_SEQ * xstride);   // [KS][16][2r]: partial k_a | v_a
  float* qa = kv_a + KS * E1_SEQ * 2 * r;                          // [G][r + 1]
  float* pg = qa + G * (r + 1);                                    // [16][G]
  int* has = reinterpret_cast<int*>(pg + E1_SEQ * G);              // [16]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nblk = (B + E1_SEQ - 1) / E1_SEQ;
  const int li = blockIdx.x / nblk;
  const int b0 = (blockIdx.x - li * nblk) * E1_SEQ;
  const int l = a.l0 + li;
  const int b = b0 + warp;                           // this warp's sequence
  const size_t lb = (size_t)l * B + b;
  const size_t ob = (size_t)li * B + b;
  const int vpr = d_kv >> 3;                         // 16-byte vectors per token row (all KV heads)
  const int gr = G * r;
  float* S = p.S + lb * gr;
  const int tiles_per_map = r >> 3;
  const int n_tiles = 2 * tiles_per_map;
  const int n_pairs = d_kv >> 5;                     // 32 k-values per pair of mma steps

  // ---- everything that does not depend on the ring state is requested first, in one round trip: the ring state
  //      itself, the arriving rows, the encoder flag; then Q_a and L2 prefetches of what the later phases read ----------
  int rs_head = 0, rs_count = 0, rs_sink = 0, rs_act = 0;
  long long rs_n = 0;
  uint4 nk[2], nv[2];
  const bool pre_new = APPEND && vpr <= 64 && b < B;           // arriving rows fit two vectors per lane
  if (APPEND) {
    if (lane == 0 && b < B) {
      rs_act = (a.active == nullptr) ? 1 : (int)a.active[b];
      rs_head = p.head[lb];
      rs_count = p.count[lb];
      rs_sink = p.n_sink[lb];
      rs_n = p.n_app[lb];
    }
    if (pre_new) {
      const int vph = p.D >> 3;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int v = lane + 32 * u;
        if (v < vpr) {
          const int h = v / vph, vv = v - h * vph;
          const size_t src = ((ob * p.Hkv + h) * p.D) * 2 + (size_t)vv * 16;
          nk[u] = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.k_new) + src);
          nv[u] = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.v_new) + src);
        }
      }
    }
  }
  const bool enc_on = p.encode_enabled && p.enc_set[l];
  if (enc_on) {
    for (int i = tid; i < gr; i += E1_THREADS) {
      const int gi = i / r;
      qa[gi * (r + 1) + (i - gi * r)] = p.Qa[(size_t)l * gr + i];
    }
    if (b < B)
      for (int i = lane; i * 32 < gr; i += 32) e1_prefetch_l2(S + i * 32);
    for (int item = warp; item < n_tiles * KS; item += E1_WARPS) {
      const int tile = item % n_tiles, ks = item / n_tiles;
      const int mat = tile >= tiles_per_map ? 1 : 0;
      const int j0 = (tile - mat * tiles_per_map) * 8;
      const int s_lo = ks * n_pairs / KS, s_hi = (ks + 1) * n_pairs / KS;
      const __nv_bfloat16* w0 = reinterpret_cast<const __nv_bfloat16*>(mat ? p.Wv : p.Wk) + (size_t)l * r * d_kv;
      const int lines = (s_hi - s_lo + 1) / 2;       // 64 bytes per pair
      for (int i = lane; i < 8 * lines; i += 32)
        e1_prefetch_l2(w0 + (size_t)(j0 + (i & 7)) * d_kv + (size_t)s_lo * 32 + (size_t)(i >> 3) * 64);
    }
  }

  // ---- phase A: the sequence's evicted row -> shared memory (+ staging), the arriving row -> ring ---------------
  int m = 0;
  if (APPEND) {
    int ev_slot = 0, new_slot = -1;
    if (lane == 0 && b < B) {
      if (rs_act != 0) {
        int head = rs_head, count = rs_count;
        const long long n = rs_n;
        const int ns = rs_sink;                      // pinned prompt entries; the ring runs over slots [ns, W)
        const int cap = W - ns;
        if (ns < 0 || cap < 1 || head < 0 || head >= cap || count < 0 || count > cap) {
          atomicOr(p.status, PTENC_ST_BAD_INDEX);
        } else {
          long long first = -1;
          if (count == cap) {                        // full: the oldest token leaves, its slot is reused at once
            m = 1;
            ev_slot = ns + head;
            first = n - count;
            head = head + 1 == cap ? 0 : head + 1;
            count -= 1;
          }
          new_slot = head + count;
          if (new_slot >= cap) new_slot -= cap;
          new_slot += ns;
          p.head[lb] = head;
          p.count[lb] = count + 1;
          p.n_app[lb] = n + 1;
          p.n_staged[lb] = m;
          p.evict_first[lb] = first;
        }
      } else {
        p.n_staged[lb] = 0;
        p.evict_first[lb] = -1;
      }
    }
    m = __shfl_sync(0xffffffffu, m, 0);
    ev_slot = __shfl_sync(0xffffffffu, ev_slot, 0);
    new_slot = __shfl_sync(0xffffffffu, new_slot, 0);
    const int vph = p.D >> 3;                        // vectors per (token, head) row
    for (int v = lane; v < vpr; v += 32) {
      const int h = v / vph, vv = v - h * vph;
      uint4 k4 = make_uint4(0u, 0u, 0u, 0u), v4 = k4;
      if (m) {
        const size_t src = (((lb * p.Hkv + h) * W + ev_slot) * p.D) * 2 + (size_t)vv * 16;
        k4 = *reinterpret_cast<const uint4*>(p.K + src);
        v4 = *reinterpret_cast<const uint4*>(p.V + src);
        const size_t dst = (lb * d_kv) * 2 + (size_t)v * 16;            // E = 1: one staged row per sequence
        *reinterpret_cast<uint4*>(p.stageK + dst) = k4;
        *reinterpret_cast<uint4*>(p.stageV + dst) = v4;
      }
      *reinterpret_cast<uint4*>(xk + warp * xstride + v * 16) = k4;
      *reinterpret_cast<uint4*>(xv + warp * xstride + v * 16) = v4;
      if (new_slot >= 0) {
        // the same lane read this address above when the ring was full, so the read precedes the write
        const size_t dst = (((lb * p.Hkv + h) * W + new_slot) * p.D) * 2 + (size_t)vv * 16;
        if (pre_new) {
          const int u = v >> 5;                      // v = lane + 32 u, u < 2
          *reinterpret_cast<uint4*>(p.K + dst) = u == 0 ? nk[0] : nk[1];
          *reinterpret_cast<uint4*>(p.V + dst) = u == 0 ? nv[0] : nv[1];
        } else {
          const size_t src = ((ob * p.Hkv + h) * p.D) * 2 + (size_t)vv * 16;
          *reinterpret_cast<uint4*>(p.K + dst) =
              *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.k_new) + src);
          *reinterpret_cast<uint4*>(p.V + dst) =
              *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.v_new) + src);
        }
      }
    }
  } else {
    if (b < B) m = (a.Ke == nullptr) ? p.n_staged[lb] : a.n_ev[ob];
    m = m > 0 ? 1 : 0;
    const __nv_bfloat16* rk = (a.Ke == nullptr) ? reinterpret_cast<const __nv_bfloat16*>(p.stageK) + lb * d_kv
                                                : a.Ke + ob * d_kv;
    const __nv_bfloat16* rv = (a.Ke == nullptr) ? reinterpret_cast<const __nv_bfloat16*>(p.stageV) + lb * d_kv
                                                : a.Ve + ob * d_kv;
    for (int v = lane; v < vpr; v += 32) {
      uint4 k4 = make_uint4(0u, 0u, 0u, 0u), v4 = k4;
      if (m && enc_on) {
        k4 = *reinterpret_cast<const uint4*>(rk + (size_t)v * 8);
        v4 = *reinterpret_cast<const uint4*>(rv + (size_t)v * 8);
      }
      *reinterpret_cast<uint4*>(xk + warp * xstride + v * 16) = k4;
      *reinterpret_cast<uint4*>(xv + warp * xstride + v * 16) = v4;
    }
  }
  const bool mine = enc_on && m > 0;
  if (lane == 0) has[warp] = mine ? 1 : 0;

  constexpr int NB = 32 / RJ;                        // state rows per batch: 32 registers per lane
  if (__syncthreads_or(mine ? 1 : 0) == 0) return;   // also orders phase A's shared-memory writes

  // ---- k_a = X_k W^a_K^T, v_a = X_v W^a_V^T : 2r/8 column tiles of 8, each split KS ways along d_kv ------------------
  {
    const __nv_bfloat16* Wk = reinterpret_cast<const __nv_bfloat16*>(p.Wk) + (size_t)l * r * d_kv;
    const __nv_bfloat16* Wv = reinterpret_cast<const __nv_bfloat16*>(p.Wv) + (size_t)l * r * d_kv;
    const int qrow = lane >> 2, qcol = lane & 3;
    for (int item = warp; item < n_tiles * KS; item += E1_WARPS) {
      const int tile = item % n_tiles, ks = item / n_tiles;
      const int mat = tile >= tiles_per_map ? 1 : 0;
      const int j0 = (tile - mat * tiles_per_map) * 8;
      const int s_lo = ks * n_pairs / KS, s_hi = (ks + 1) * n_pairs / KS;
      const __nv_bfloat16* wrow = (mat ? Wv : Wk) + (size_t)(j0 + qrow) * d_kv + qcol * 8;
      const uint8_t* xa = (mat ? xv : xk) + qrow * xstride + qcol * 16;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
      for (int s0 = s_lo; s0 < s_hi; s0 += 8) {
        uint4 bw[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (s0 + u < s_hi) bw[u] = __ldg(reinterpret_cast<const uint4*>(wrow + (size_t)(s0 + u) * 32));
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          if (s0 + u < s_hi) {
            const uint4 lo = *reinterpret_cast<const uint4*>(xa + (s0 + u) * 64);
            const uint4 hi = *reinterpret_cast<const uint4*>(xa + 8 * xstride + (s0 + u) * 64);
            e1_mma(c, lo.x, hi.x, lo.y, hi.y, bw[u].x, bw[u].y);
            e1_mma(c, lo.z, hi.z, lo.w, hi.w, bw[u].z, bw[u].w);
          }
        }
      }
      float* dst = kv_a + (size_t)ks * E1_SEQ * 2 * r + mat * r + j0 + 2 * qcol;
      dst[qrow * 2 * r] = c[0];
      dst[qrow * 2 * r + 1] = c[1];
      dst[(qrow + 8) * 2 * r] = c[2];
      dst[(qrow + 8) * 2 * r + 1] = c[3];
    }
  }
  __syncthreads();
  if (KS > 1) {                                      // sum the partial projections into the first copy
    for (int i = tid; i < E1_SEQ * 2 * r; i += E1_THREADS) {
      float s = kv_a[i];
      for (int ks = 1; ks < KS; ++ks) s += kv_a[(size_t)ks * E1_SEQ * 2 * r + i];
      kv_a[i] = s;
    }
    __syncthreads();
  }

  // ---- p = Q_a k_a ----------------------------------------------------------------------------------------------------
  for (int idx = tid; idx < E1_SEQ * G; idx += E1_THREADS) {
    const int row = idx / G, gi = idx - row * G;
    float sacc = 0.f;
    for (int j = 0; j < r; ++j) sacc = fmaf(qa[gi * (r + 1) + j], kv_a[row * 2 * r + j], sacc);
    pg[idx] = sacc;
  }
  __syncthreads();

  // ---- S <- Normalize(S + p v_a^T): one warp per sequence, a state row across the lanes ------------------------------
  if (!mine) return;
  const float* va = kv_a + warp * 2 * r + r;
  float total = 0.f;
  for (int g0 = 0; g0 < G; g0 += NB) {
    float st[NB][RJ];
#pragma unroll
    for (int u = 0; u < NB; ++u)
#pragma unroll
      for (int jj = 0; jj < RJ; ++jj) {
        const int gi = g0 + u, j = lane + 32 * jj;
        st[u][jj] = (gi < G && j < r) ? S[gi * r + j] : 0.f;
      }
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      const int gi = g0 + u;
      if (gi < G) {
        const float pw = pg[warp * G + gi];
        float ss = 0.f;
#pragma unroll
        for (int jj = 0; jj < RJ; ++jj) {
          const int j = lane + 32 * jj;
          if (j < r) {
            st[u][jj] = fmaf(pw, va[j], st[u][jj]);
            ss = fmaf(st[u][jj], st[u][jj], ss);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        total += ss;
        const float sc = (p.norm_mode == PTENC_NORM_ROW_L2) ? rsqrtf(fmaxf(ss, 1e-24f)) : 1.f;   // 1 / max(|row|, 1e-12)
#pragma unroll
        for (int jj = 0; jj < RJ; ++jj) {
          const int j = lane + 32 * jj;
          if (j < r) S[gi * r + j] = st[u][jj] * sc;
        }
      }
    }
  }
  if (p.norm_mode == PTENC_NORM_FROBENIUS) {
    // the un-normalised sum was stored above; every lane rescales the elements it wrote itself
    const float sc = 1.f / fmaxf(sqrtf(total), 1e-12f);
    for (int gi = 0; gi < G; ++gi)
      for (int j = lane; j < r; j += 32) S[gi * r + j] *= sc;
  }
}

template <bool APPEND, int RJ>
cudaError_t e1_launch_t(ptenc_cache* c, int nl, const E1Args& a, cudaStream_t st) {
  const PtencDev& p = c->dev;
  const size_t smem = e1_smem_bytes(p.G, p.r, p.d_kv);
  static bool attr_done[PTENC_MAX_DEVICES] = {};
  if (ptenc_first_use(attr_done, c->cfg.device)) {
    cudaError_t e = cudaFuncSetAttribute(k_step_e1<APPEND, RJ>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         200 * 1024);
    if (e != cudaSuccess) return e;
  }
  const int nblk = (p.B + E1_SEQ - 1) / E1_SEQ;
  k_step_e1<APPEND, RJ><<<nl * nblk, E1_THREADS, smem, st>>>(p, a);
  c->launches++;
  return cudaGetLastError();
}

template <bool APPEND>
cudaError_t e1_launch(ptenc_cache* c, int nl, const E1Args& a, cudaStream_t st) {
  const int rj = (c->dev.r + 31) / 32;
  if (rj == 1) return e1_launch_t<APPEND, 1>(c, nl, a, st);
  if (rj == 2) return e1_launch_t<APPEND, 2>(c, nl, a, st);
  return e1_launch_t<APPEND, 4>(c, nl, a, st);
}

}  // namespace

// bf16 storage, one row per sequence, r a multiple of 8 (column tiles of the mma), d_kv a multiple of 32.
bool ptenc_step_e1_usable(const ptenc_cache* c, const void* Ke, int m_max) {
  const PtencDev& p = c->dev;
  if (c->cfg.dtype != PTENC_DTYPE_BF16 || (p.r & 7) != 0 || (p.d_kv & 31) != 0) return false;
  if (Ke == nullptr ? p.E != 1 : m_max != 1) return false;
  return e1_smem_bytes(p.G, p.r, p.d_kv) <= 200 * 1024;
}

cudaError_t ptenc_launch_step_e1(ptenc_cache* c, int l0, int nl, bool append, const void* k_new, const void* v_new,
                                 const uint8_t* active, const void* Ke, const void* Ve, const int32_t* n_ev,
                                 int m_max, cudaStream_t st) {
  (void)m_max;
  E1Args a;
  a.l0 = l0;
  a.k_new = static_cast<const __nv_bfloat16*>(k_new);
  a.v_new = static_cast<const __nv_bfloat16*>(v_new);
  a.active = active;
  a.Ke = static_cast<const __nv_bfloat16*>(Ke);
  a.Ve = static_cast<const __nv_bfloat16*>(Ve);
  a.n_ev = n_ev;
  a.k_split = e1_k_split(c->dev.r);
  return append ? e1_launch<true>(c, nl, a, st) : e1_launch<false>(c, nl, a, st);
}
