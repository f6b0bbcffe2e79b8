// Progressive encoder (step a3) and its set-up, Sec. 3.3, Eq. (3):
//   S' = ((W^a_Q q_g)(W^a_K K_e)^T)(W^a_V V_e),   S <- Normalize(S + S'),
// and the bootstrap S_0 built the same way from the global tokens' keys and values.
// The evicted rows of one sequence are folded as a sum of rank-1 terms (Q_a k_a,i) v_a,i^T, which equals
// the bracketed product exactly up to summation order; nothing is scaled and there is no softmax.
#include "ptenc_internal.h"

namespace {

constexpr int ENC_THREADS = 256;

template <typename T> struct Vec16;
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void load16(const T* ptr, float (&out)[Vec16<T>::N]) {
  uint4 raw = *reinterpret_cast<const uint4*>(ptr);
  const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
  for (int i = 0; i < Vec16<T>::N; ++i) out[i] = ptenc_to_float(e[i]);
}

// Q_a[g][j] = sum_d q_g[g][d] * W^a_Q[j][d].  One warp per output.
template <typename T>
__global__ void __launch_bounds__(ENC_THREADS)
k_latent_queries(PtencDev p, int layer, const T* __restrict__ Wq, const T* __restrict__ qg) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= p.G * p.r) return;
  const int gi = warp / p.r, j = warp - gi * p.r;
  constexpr int N = Vec16<T>::N;
  float s = 0.f;
  for (int d = lane * N; d < p.d_q; d += 32 * N) {
    float a[N], w[N];
    load16(qg + (size_t)gi * p.d_q + d, a);
    load16(Wq + (size_t)j * p.d_q + d, w);
#pragma unroll
    for (int i = 0; i < N; ++i) s = fmaf(a[i], w[i], s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) p.Qa[((size_t)layer * p.G + gi) * p.r + j] = s;
}

// mode 0: fold `m` rows into S[l][b] and normalise.   grid = nl * B
// mode 1: S0[l] = context state of the G global rows (no base, no normalise).  grid = 1
template <typename T>
__global__ void __launch_bounds__(ENC_THREADS)
k_encode_rows(PtencDev p, int l0, const T* __restrict__ Ke, const T* __restrict__ Ve,
              const int32_t* __restrict__ n_ev, int m_max, int mode) {
  extern __shared__ float sm[];
  const int G = p.G, r = p.r, d_kv = p.d_kv;
  float* xk = sm;
  float* xv = xk + d_kv;
  float* ka = xv + d_kv;           // ka[0..r), va = ka + r
  float* pg = ka + 2 * r;
  float* qa = pg + G;
  float* acc = qa + G * r;
  float* red = acc + G * r;        // G + 1

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  int l, b, m;
  const T *rowsK, *rowsV;
  if (mode == 1) {
    l = l0; b = 0; m = G;
    rowsK = Ke; rowsV = Ve;
  } else {
    const int li = blockIdx.x / p.B;
    b = blockIdx.x - li * p.B;
    l = l0 + li;
    if (!p.encode_enabled || !p.enc_set[l]) return;
    if (Ke == nullptr) {
      m = p.n_staged[(size_t)l * p.B + b];
      rowsK = reinterpret_cast<const T*>(p.stageK) + ((size_t)l * p.B + b) * p.E * d_kv;
      rowsV = reinterpret_cast<const T*>(p.stageV) + ((size_t)l * p.B + b) * p.E * d_kv;
    } else {
      m = n_ev[(size_t)li * p.B + b];
      if (m > m_max) m = m_max;
      rowsK = Ke + ((size_t)li * p.B + b) * m_max * d_kv;
      rowsV = Ve + ((size_t)li * p.B + b) * m_max * d_kv;
    }
    if (m <= 0) return;
  }
  const T* Wk = reinterpret_cast<const T*>(p.Wk) + (size_t)l * r * d_kv;
  const T* Wv = reinterpret_cast<const T*>(p.Wv) + (size_t)l * r * d_kv;
  const int gr = G * r;
  for (int i = tid; i < gr; i += blockDim.x) {
    qa[i] = p.Qa[(size_t)l * gr + i];
    acc[i] = 0.f;
  }
  constexpr int N = Vec16<T>::N;

  for (int row = 0; row < m; ++row) {
    __syncthreads();
    for (int d = tid; d < d_kv; d += blockDim.x) {
      xk[d] = ptenc_to_float(rowsK[(size_t)row * d_kv + d]);
      xv[d] = ptenc_to_float(rowsV[(size_t)row * d_kv + d]);
    }
    __syncthreads();
    // k_a = W^a_K k_e, v_a = W^a_V v_e : 2r dot products of length d_kv, one warp each
    for (int j = warp; j < 2 * r; j += nwarps) {
      const T* wrow = (j < r) ? (Wk + (size_t)j * d_kv) : (Wv + (size_t)(j - r) * d_kv);
      const float* x = (j < r) ? xk : xv;
      float s = 0.f;
      for (int d = lane * N; d < d_kv; d += 32 * N) {
        float w[N];
        load16(wrow + d, w);
#pragma unroll
        for (int i = 0; i < N; ++i) s = fmaf(w[i], x[d + i], s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) ka[j] = s;
    }
    __syncthreads();
    // p = Q_a k_a
    for (int gi = tid; gi < G; gi += blockDim.x) {
      float s = 0.f;
      for (int j = 0; j < r; ++j) s = fmaf(qa[gi * r + j], ka[j], s);
      pg[gi] = s;
    }
    __syncthreads();
    // S' += p v_a^T
    for (int i = tid; i < gr; i += blockDim.x) {
      const int gi = i / r, j = i - gi * r;
      acc[i] = fmaf(pg[gi], ka[r + j], acc[i]);
    }
  }
  __syncthreads();

  if (mode == 1) {
    for (int i = tid; i < gr; i += blockDim.x) p.S0[(size_t)l * gr + i] = acc[i];
    return;
  }
  float* S = p.S + ((size_t)l * p.B + b) * gr;
  for (int i = tid; i < gr; i += blockDim.x) acc[i] += S[i];
  __syncthreads();
  if (p.norm_mode == PTENC_NORM_ROW_L2) {
    for (int gi = warp; gi < G; gi += nwarps) {
      float s = 0.f;
      for (int j = lane; j < r; j += 32) s = fmaf(acc[gi * r + j], acc[gi * r + j], s);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) red[gi] = 1.f / fmaxf(sqrtf(s), 1e-12f);
    }
    __syncthreads();
    for (int i = tid; i < gr; i += blockDim.x) S[i] = acc[i] * red[i / r];
  } else if (p.norm_mode == PTENC_NORM_FROBENIUS) {
    for (int gi = warp; gi < G; gi += nwarps) {
      float s = 0.f;
      for (int j = lane; j < r; j += 32) s = fmaf(acc[gi * r + j], acc[gi * r + j], s);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) red[gi] = s;
    }
    __syncthreads();
    if (tid == 0) {
      float s = 0.f;
      for (int gi = 0; gi < G; ++gi) s += red[gi];
      red[G] = 1.f / fmaxf(sqrtf(s), 1e-12f);
    }
    __syncthreads();
    for (int i = tid; i < gr; i += blockDim.x) S[i] = acc[i] * red[G];
  } else {
    for (int i = tid; i < gr; i += blockDim.x) S[i] = acc[i];
  }
}

// ---------------------------------------------------------------------------------------------------------------
// One evicted token per sequence (E = 1, the ring-per-step mode), bf16 storage: the projections of a block of 16
// sequences of one layer are one small matrix product X [16, d_kv] x W^T [d_kv, r] per map, done with warp-level
// bf16 mma (fp32 accumulate) so that the layer's weights are read once per 16 sequences instead of once per
// sequence.  Each lane fetches 8 consecutive k-values of its A row (shared memory) and of its B row (W^a, from L2)
// with one 16-byte load and feeds them to two mma steps; the contraction index is permuted the same way on both
// operands, which leaves the sum unchanged.  Then p = Q_a k_a, S + p v_a^T, Normalize, all in fp32.
// ---------------------------------------------------------------------------------------------------------------
constexpr int ES_SEQ = 16;
constexpr int ES_THREADS = 256;
constexpr int ES_WARPS = ES_THREADS / 32;

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__host__ __device__ inline size_t encode_step_smem(int G, int r, int d_kv) {
  const size_t xstride = (size_t)d_kv * 2 + 64;
  return 2 * ES_SEQ * xstride + sizeof(float) * ((size_t)ES_SEQ * 2 * r + (size_t)G * (r + 1) + (size_t)ES_SEQ * G) +
         ES_SEQ * sizeof(int);
}

__global__ void __launch_bounds__(ES_THREADS)
k_encode_step_mma(PtencDev p, int l0, const __nv_bfloat16* __restrict__ Ke, const __nv_bfloat16* __restrict__ Ve,
                  const int32_t* __restrict__ n_ev, int m_max) {
  extern __shared__ __align__(16) uint8_t es_smem[];
  const int G = p.G, r = p.r, d_kv = p.d_kv, B = p.B;
  const int xstride = d_kv * 2 + 64;                 // bytes; = 64 mod 128 keeps the 16-byte A loads conflict-free
  uint8_t* xk = es_smem;
  uint8_t* xv = xk + ES_SEQ * xstride;
  float* kv_a = reinterpret_cast<float*>(xv + ES_SEQ * xstride);   // [16][2r]: k_a | v_a of each sequence
  float* qa = kv_a + ES_SEQ * 2 * r;                               // [G][r + 1]
  float* pg = qa + G * (r + 1);                                    // [16][G]
  int* has = reinterpret_cast<int*>(pg + ES_SEQ * G);              // [16]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nblk = (B + ES_SEQ - 1) / ES_SEQ;
  const int li = blockIdx.x / nblk;
  const int b0 = (blockIdx.x - li * nblk) * ES_SEQ;
  const int l = l0 + li;
  if (!p.encode_enabled || !p.enc_set[l]) return;

  int mine = 0;
  if (tid < ES_SEQ) {
    const int b = b0 + tid;
    if (b < B) mine = (Ke == nullptr) ? p.n_staged[(size_t)l * B + b] : min(n_ev[(size_t)li * B + b], m_max);
    has[tid] = mine > 0 ? 1 : 0;
  }
  if (__syncthreads_or(mine > 0) == 0) return;

  // ---- the evicted rows of the 16 sequences (zero rows where nothing was evicted) -----------------------------------
  const int vpr = d_kv >> 3;                         // 16-byte vectors per row
  for (int idx = tid; idx < ES_SEQ * vpr; idx += ES_THREADS) {
    const int row = idx / vpr, v = idx - row * vpr;
    uint4 k4 = make_uint4(0u, 0u, 0u, 0u), v4 = k4;
    if (has[row]) {
      const int b = b0 + row;
      const size_t src = (Ke == nullptr) ? ((size_t)l * B + b) * p.E * d_kv : ((size_t)li * B + b) * m_max * d_kv;
      const __nv_bfloat16* rk = (Ke == nullptr) ? reinterpret_cast<const __nv_bfloat16*>(p.stageK) : Ke;
      const __nv_bfloat16* rv = (Ke == nullptr) ? reinterpret_cast<const __nv_bfloat16*>(p.stageV) : Ve;
      k4 = *reinterpret_cast<const uint4*>(rk + src + (size_t)v * 8);
      v4 = *reinterpret_cast<const uint4*>(rv + src + (size_t)v * 8);
    }
    *reinterpret_cast<uint4*>(xk + row * xstride + v * 16) = k4;
    *reinterpret_cast<uint4*>(xv + row * xstride + v * 16) = v4;
  }
  const int gr = G * r;
  for (int i = tid; i < gr; i += ES_THREADS) {
    const int gi = i / r;
    qa[gi * (r + 1) + (i - gi * r)] = p.Qa[(size_t)l * gr + i];
  }
  __syncthreads();

  // ---- k_a = X_k W^a_K^T, v_a = X_v W^a_V^T : 2r/8 column tiles of 8, spread over the warps ------------------------
  {
    const __nv_bfloat16* Wk = reinterpret_cast<const __nv_bfloat16*>(p.Wk) + (size_t)l * r * d_kv;
    const __nv_bfloat16* Wv = reinterpret_cast<const __nv_bfloat16*>(p.Wv) + (size_t)l * r * d_kv;
    const int tiles_per_map = r >> 3;
    const int n_pairs = d_kv >> 5;                   // 32 k-values per pair of mma steps
    const int qrow = lane >> 2, qcol = lane & 3;
    for (int tile = warp; tile < 2 * tiles_per_map; tile += ES_WARPS) {
      const int mat = tile >= tiles_per_map ? 1 : 0;
      const int j0 = (tile - mat * tiles_per_map) * 8;
      const __nv_bfloat16* wrow = (mat ? Wv : Wk) + (size_t)(j0 + qrow) * d_kv + qcol * 8;
      const uint8_t* xa = (mat ? xv : xk) + qrow * xstride + qcol * 16;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
      for (int s0 = 0; s0 < n_pairs; s0 += 8) {
        uint4 bw[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (s0 + u < n_pairs) bw[u] = __ldg(reinterpret_cast<const uint4*>(wrow + (size_t)(s0 + u) * 32));
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          if (s0 + u < n_pairs) {
            const uint4 lo = *reinterpret_cast<const uint4*>(xa + (s0 + u) * 64);
            const uint4 hi = *reinterpret_cast<const uint4*>(xa + 8 * xstride + (s0 + u) * 64);
            mma_bf16_16816(c, lo.x, hi.x, lo.y, hi.y, bw[u].x, bw[u].y);
            mma_bf16_16816(c, lo.z, hi.z, lo.w, hi.w, bw[u].z, bw[u].w);
          }
        }
      }
      float* dst = kv_a + mat * r + j0 + 2 * qcol;
      dst[qrow * 2 * r] = c[0];
      dst[qrow * 2 * r + 1] = c[1];
      dst[(qrow + 8) * 2 * r] = c[2];
      dst[(qrow + 8) * 2 * r + 1] = c[3];
    }
  }
  __syncthreads();

  // ---- p = Q_a k_a ------------------------------------------------------------------------------------------------
  for (int idx = tid; idx < ES_SEQ * G; idx += ES_THREADS) {
    const int row = idx / G, gi = idx - row * G;
    float sacc = 0.f;
    for (int j = 0; j < r; ++j) sacc = fmaf(qa[gi * (r + 1) + j], kv_a[row * 2 * r + j], sacc);
    pg[idx] = sacc;
  }
  __syncthreads();

  // ---- S <- Normalize(S + p v_a^T): a warp per sequence, a state row per 32 lanes ------------------------------------
  const int jper = (r + 31) >> 5;                    // <= 4 elements of a row per lane
  for (int row = warp; row < ES_SEQ; row += ES_WARPS) {
    if (!has[row]) continue;
    float* S = p.S + ((size_t)l * B + b0 + row) * gr;
    const float* va = kv_a + row * 2 * r + r;
    float total = 0.f;
    for (int g0 = 0; g0 < G; g0 += 8) {
      float val[8][4];
#pragma unroll
      for (int u = 0; u < 8; ++u)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int gi = g0 + u, j = lane + 32 * jj;
          val[u][jj] = (gi < G && jj < jper && j < r) ? S[gi * r + j] : 0.f;
        }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int gi = g0 + u;
        if (gi >= G) break;
        const float pw = pg[row * G + gi];
        float ss = 0.f;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int j = lane + 32 * jj;
          if (jj < jper && j < r) {
            val[u][jj] = fmaf(pw, va[j], val[u][jj]);
            ss = fmaf(val[u][jj], val[u][jj], ss);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        total += ss;
        const float sc = (p.norm_mode == PTENC_NORM_ROW_L2) ? 1.f / fmaxf(sqrtf(ss), 1e-12f) : 1.f;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int j = lane + 32 * jj;
          if (jj < jper && j < r) S[gi * r + j] = val[u][jj] * sc;
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
}

// S[l][b] = S0[l] for every b; zero_s0 != 0 first clears S0[l].
__global__ void k_broadcast_state(PtencDev p, int layer, int zero_s0) {
  const int gr = p.G * p.r;
  const int b = blockIdx.x;
  for (int i = threadIdx.x; i < gr; i += blockDim.x) {
    float v = zero_s0 ? 0.f : p.S0[(size_t)layer * gr + i];
    p.S[((size_t)layer * p.B + b) * gr + i] = v;
  }
  if (b == 0 && threadIdx.x == 0) p.enc_set[layer] = 1;
}

__global__ void k_zero_s0(PtencDev p, int layer) {
  const int gr = p.G * p.r;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < gr; i += gridDim.x * blockDim.x)
    p.S0[(size_t)layer * gr + i] = 0.f;
}

size_t encode_smem(const PtencDev& p) {
  return sizeof(float) * (size_t)(2 * p.d_kv + 2 * p.r + p.G + 2 * p.G * p.r + p.G + 1);
}

template <typename T>
cudaError_t launch_encode_t(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve,
                            const int32_t* n_ev, int m_max, int mode, cudaStream_t st) {
  const size_t smem = encode_smem(c->dev);
  static bool attr_done[2] = {false, false};
  const int ti = sizeof(T) == 4 ? 0 : 1;
  if (!attr_done[ti] && smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k_encode_rows<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[ti] = true;
  }
  const int grid = mode == 1 ? 1 : nl * c->cfg.batch;
  k_encode_rows<T><<<grid, ENC_THREADS, smem, st>>>(c->dev, l0, (const T*)Ke, (const T*)Ve, n_ev, m_max, mode);
  c->launches++;
  return cudaGetLastError();
}

// The one-row-per-sequence tensor-core kernel covers bf16 storage with r a multiple of 8 and d_kv a multiple of 32.
bool encode_step_usable(const ptenc_cache* c, const void* Ke, int m_max) {
  const PtencDev& p = c->dev;
  if (c->cfg.dtype != PTENC_DTYPE_BF16 || (p.r & 7) != 0 || (p.d_kv & 31) != 0) return false;
  if (Ke == nullptr ? p.E != 1 : m_max != 1) return false;
  return encode_step_smem(p.G, p.r, p.d_kv) <= 160 * 1024;
}

cudaError_t launch_encode_step(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve, const int32_t* n_ev,
                               int m_max, cudaStream_t st) {
  const PtencDev& p = c->dev;
  const size_t smem = encode_step_smem(p.G, p.r, p.d_kv);
  static bool attr_done = false;
  if (!attr_done && smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k_encode_step_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  const int nblk = (p.B + ES_SEQ - 1) / ES_SEQ;
  k_encode_step_mma<<<nl * nblk, ES_THREADS, smem, st>>>(p, l0, (const __nv_bfloat16*)Ke, (const __nv_bfloat16*)Ve,
                                                         n_ev, m_max);
  c->launches++;
  return cudaGetLastError();
}

}  // namespace

cudaError_t ptenc_launch_encode(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve,
                                const int32_t* n_ev, int m_max, cudaStream_t st) {
  if (encode_step_usable(c, Ke, m_max)) return launch_encode_step(c, l0, nl, Ke, Ve, n_ev, m_max, st);
  // chunks of evicted tokens: the projections are dense contractions -> tensor cores
  if (c->tc_encode && (Ke == nullptr ? c->dev.E : m_max) >= 2 &&
      (Ke == nullptr || (long long)nl * c->cfg.batch * m_max >= 128))
    return ptenc_launch_encode_tc(c, l0, nl, Ke, Ve, n_ev, m_max, st);
  if (c->cfg.dtype == PTENC_DTYPE_FP32) return launch_encode_t<float>(c, l0, nl, Ke, Ve, n_ev, m_max, 0, st);
  return launch_encode_t<__nv_bfloat16>(c, l0, nl, Ke, Ve, n_ev, m_max, 0, st);
}

cudaError_t ptenc_launch_set_encoder(ptenc_cache* c, int layer, const void* Wq, const void* qg,
                                     const void* kg, const void* vg, cudaStream_t st) {
  const PtencDev& p = c->dev;
  const int warps = p.G * p.r;
  const int blocks = (warps * 32 + ENC_THREADS - 1) / ENC_THREADS;
  cudaError_t e;
  if (c->cfg.dtype == PTENC_DTYPE_FP32)
    k_latent_queries<float><<<blocks, ENC_THREADS, 0, st>>>(p, layer, (const float*)Wq, (const float*)qg);
  else
    k_latent_queries<__nv_bfloat16><<<blocks, ENC_THREADS, 0, st>>>(p, layer, (const __nv_bfloat16*)Wq,
                                                                   (const __nv_bfloat16*)qg);
  c->launches++;
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  const bool have_global = (kg != nullptr && vg != nullptr);
  if (have_global) {
    if (c->cfg.dtype == PTENC_DTYPE_FP32)
      e = launch_encode_t<float>(c, layer, 1, kg, vg, nullptr, p.G, 1, st);
    else
      e = launch_encode_t<__nv_bfloat16>(c, layer, 1, kg, vg, nullptr, p.G, 1, st);
    if (e != cudaSuccess) return e;
  } else {
    k_zero_s0<<<4, 256, 0, st>>>(p, layer);
    c->launches++;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  k_broadcast_state<<<p.B, 256, 0, st>>>(p, layer, 0);
  c->launches++;
  return cudaGetLastError();
}
