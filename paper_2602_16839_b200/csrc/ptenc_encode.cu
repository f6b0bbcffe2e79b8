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
  static bool attr_done[PTENC_MAX_DEVICES] = {};          // one per instantiation of this template
  if (smem > 48 * 1024 && ptenc_first_use(attr_done, c->cfg.device)) {
    cudaError_t e = cudaFuncSetAttribute(k_encode_rows<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
  }
  const int grid = mode == 1 ? 1 : nl * c->cfg.batch;
  k_encode_rows<T><<<grid, ENC_THREADS, smem, st>>>(c->dev, l0, (const T*)Ke, (const T*)Ve, n_ev, m_max, mode);
  c->launches++;
  return cudaGetLastError();
}

}  // namespace

cudaError_t ptenc_launch_encode(ptenc_cache* c, int l0, int nl, const void* Ke, const void* Ve,
                                const int32_t* n_ev, int m_max, cudaStream_t st) {
  // one evicted token per sequence: a warp per sequence
  if (ptenc_step_e1_usable(c, Ke, m_max)) return ptenc_launch_encode_e1(c, l0, nl, Ke, Ve, n_ev, st);
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
