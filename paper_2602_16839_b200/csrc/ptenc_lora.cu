// Dynamic weight update (Sec. 3.3, Eq. (3)): Delta W = A S_e B, theta' = theta + Delta W, recomputed whenever the
// state changes.  Delta W is never formed: for the one token a sequence decodes per step,
//   y_b += Delta W_b x_b = A (S_b (B x_b)),
// three thin products per sequence (r x d_in, G x r, d_out x G).  Each sequence has its own state, so this is a
// batch of tiny products; the only sizeable traffic is A and B, which a CTA reads once for a block of sequences.
// fp32 accumulation throughout; x, y, A, B in the storage dtype.
#include "ptenc_internal.h"

namespace {

constexpr int LR_SEQ = 8;            // sequences per CTA
constexpr int LR_THREADS = 256;
constexpr int LR_WARPS = LR_THREADS / 32;

template <typename T> struct LrVec;
template <> struct LrVec<float> { static constexpr int N = 4; };
template <> struct LrVec<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void lr_load16(const T* ptr, float (&out)[LrVec<T>::N]) {
  const uint4 raw = *reinterpret_cast<const uint4*>(ptr);
  const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
  for (int i = 0; i < LrVec<T>::N; ++i) out[i] = ptenc_to_float(e[i]);
}

// grid = nl * ceil(B / LR_SEQ).  A [nl][d_out][G], Bm [nl][r][d_in], x [nl][B][d_in], y [nl][B][d_out].
template <typename T>
__global__ void __launch_bounds__(LR_THREADS)
k_lora_apply(PtencDev p, int l0, const T* __restrict__ A, const T* __restrict__ Bm, const T* __restrict__ x,
             T* __restrict__ y, const uint8_t* __restrict__ active, int d_in, int d_out) {
  extern __shared__ __align__(16) float lr_smem[];
  const int G = p.G, r = p.r, B = p.B;
  float* u = lr_smem;                    // [LR_SEQ][r]   B x
  float* w = u + LR_SEQ * r;             // [LR_SEQ][G]   S (B x)
  float* Ss = lr_smem + ((LR_SEQ * (r + G) + 3) & ~3);                      // [LR_SEQ][G][r + 1] the block's states
  T* xs = reinterpret_cast<T*>(Ss + ((LR_SEQ * G * (r + 1) + 3) & ~3));     // [LR_SEQ][d_in] the block's inputs
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nblk = (B + LR_SEQ - 1) / LR_SEQ;
  const int li = blockIdx.x / nblk;
  const int b0 = (blockIdx.x - li * nblk) * LR_SEQ;
  const int l = l0 + li;
  const int nseq = min(LR_SEQ, B - b0);
  constexpr int N = LrVec<T>::N;
  const T* Bl = Bm + (size_t)li * r * d_in;
  const T* Al = A + (size_t)li * d_out * G;
  const T* xl = x + ((size_t)li * B + b0) * d_in;
  T* yl = y + ((size_t)li * B + b0) * d_out;

  // the block's input rows and states, read once with every load in flight together
  for (int idx = tid * N; idx < nseq * d_in; idx += LR_THREADS * N)
    *reinterpret_cast<uint4*>(xs + idx) = *reinterpret_cast<const uint4*>(xl + idx);
  {
    const float* Sg = p.S + ((size_t)l * B + b0) * G * r;
    for (int idx = tid; idx < nseq * G * r; idx += LR_THREADS) {
      const int row = idx / r;
      Ss[row * (r + 1) + (idx - row * r)] = Sg[idx];
    }
  }
  __syncthreads();

  // ---- u[s][j] = <B[j,:], x_s> : a warp per row j of B, the row's values shared by the block's sequences -----------
  for (int j = warp; j < r; j += LR_WARPS) {
    float acc[LR_SEQ];
#pragma unroll
    for (int s = 0; s < LR_SEQ; ++s) acc[s] = 0.f;
    // four 16-byte loads of the row in flight per lane: the loop is bound by load latency, not by arithmetic
    for (int d0 = lane * N; d0 < d_in; d0 += 4 * 32 * N) {
      uint4 raw[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int d = d0 + q * 32 * N;
        raw[q] = d < d_in ? __ldg(reinterpret_cast<const uint4*>(Bl + (size_t)j * d_in + d)) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int d = d0 + q * 32 * N;
        if (d < d_in) {
          float bv[N];
          const T* e = reinterpret_cast<const T*>(&raw[q]);
#pragma unroll
          for (int i = 0; i < N; ++i) bv[i] = ptenc_to_float(e[i]);
#pragma unroll
          for (int s = 0; s < LR_SEQ; ++s) {
            if (s < nseq) {
              float xv[N];
              lr_load16(xs + (size_t)s * d_in + d, xv);
#pragma unroll
              for (int i = 0; i < N; ++i) acc[s] = fmaf(bv[i], xv[i], acc[s]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int s = 0; s < LR_SEQ; ++s) {
      float a = acc[s];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      if (lane == 0) u[s * r + j] = a;
    }
  }
  __syncthreads();
  // ---- w[s][g] = <S_s[g,:], u_s> ------------------------------------------------------------------------------------
  for (int idx = tid; idx < nseq * G; idx += LR_THREADS) {
    const int s = idx / G, g = idx - s * G;
    const float* Srow = Ss + (size_t)idx * (r + 1);
    float a = 0.f;
    for (int j = 0; j < r; ++j) a = fmaf(Srow[j], u[s * r + j], a);
    w[idx] = a;
  }
  __syncthreads();
  // ---- y[s][i] += <A[i,:], w_s> : a thread per output row i, consecutive threads on consecutive outputs -----------
  for (int i = tid; i < d_out; i += LR_THREADS) {
    float acc[LR_SEQ], yold[LR_SEQ];
#pragma unroll
    for (int s = 0; s < LR_SEQ; ++s) {
      acc[s] = 0.f;
      yold[s] = s < nseq ? ptenc_to_float(yl[(size_t)s * d_out + i]) : 0.f;    // in flight during the products
    }
    if ((G & (N - 1)) == 0) {                       // rows of A are whole 16-byte vectors
      for (int g = 0; g < G; g += N) {
        float av[N];
        lr_load16(Al + (size_t)i * G + g, av);
#pragma unroll
        for (int k = 0; k < N; ++k)
#pragma unroll
          for (int s = 0; s < LR_SEQ; ++s) acc[s] = fmaf(av[k], w[s * G + g + k], acc[s]);
      }
    } else {
      for (int g = 0; g < G; ++g) {
        const float av = ptenc_to_float(Al[(size_t)i * G + g]);
#pragma unroll
        for (int s = 0; s < LR_SEQ; ++s) acc[s] = fmaf(av, w[s * G + g], acc[s]);
      }
    }
#pragma unroll
    for (int s = 0; s < LR_SEQ; ++s) {
      if (s < nseq && (active == nullptr || active[b0 + s] != 0)) {
        yl[(size_t)s * d_out + i] = ptenc_from_float<T>(yold[s] + acc[s]);
      }
    }
  }
}

}  // namespace

cudaError_t ptenc_launch_lora_apply(ptenc_cache* c, int l0, int nl, const void* A, const void* Bm, const void* x,
                                    void* y, const uint8_t* active, int d_in, int d_out, cudaStream_t st) {
  const PtencDev& p = c->dev;
  const size_t smem = sizeof(float) * ((((size_t)LR_SEQ * (p.r + p.G) + 3) & ~(size_t)3) +
                                       (((size_t)LR_SEQ * p.G * (p.r + 1) + 3) & ~(size_t)3)) +
                      (size_t)LR_SEQ * d_in * p.elt;
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_lora_apply<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_lora_apply<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  const int nblk = (p.B + LR_SEQ - 1) / LR_SEQ;
  if (c->cfg.dtype == PTENC_DTYPE_FP32)
    k_lora_apply<float><<<nl * nblk, LR_THREADS, smem, st>>>(p, l0, (const float*)A, (const float*)Bm,
                                                             (const float*)x, (float*)y, active, d_in, d_out);
  else
    k_lora_apply<__nv_bfloat16><<<nl * nblk, LR_THREADS, smem, st>>>(
        p, l0, (const __nv_bfloat16*)A, (const __nv_bfloat16*)Bm, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, active,
        d_in, d_out);
  c->launches++;
  return cudaGetLastError();
}
