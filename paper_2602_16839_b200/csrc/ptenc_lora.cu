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
  extern __shared__ float lr_smem[];
  const int G = p.G, r = p.r, B = p.B;
  float* u = lr_smem;                    // [LR_SEQ][r]   B x
  float* w = u + LR_SEQ * r;             // [LR_SEQ][G]   S (B x)
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

  // ---- u[s][j] = <B[j,:], x_s> : a warp per row j of B, the row's values shared by the block's sequences -----------
  for (int j = warp; j < r; j += LR_WARPS) {
    float acc[LR_SEQ];
#pragma unroll
    for (int s = 0; s < LR_SEQ; ++s) acc[s] = 0.f;
    for (int d = lane * N; d < d_in; d += 32 * N) {
      float bv[N];
      lr_load16(Bl + (size_t)j * d_in + d, bv);
#pragma unroll
      for (int s = 0; s < LR_SEQ; ++s) {
        if (s < nseq) {
          float xv[N];
          lr_load16(xl + (size_t)s * d_in + d, xv);
#pragma unroll
          for (int i = 0; i < N; ++i) acc[s] = fmaf(bv[i], xv[i], acc[s]);
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
    const float* Srow = p.S + (((size_t)l * B + b0 + s) * G + g) * r;
    float a = 0.f;
    for (int j = 0; j < r; ++j) a = fmaf(Srow[j], u[s * r + j], a);
    w[idx] = a;
  }
  __syncthreads();
  // ---- y[s][i] += <A[i,:], w_s> : a thread per output row i, consecutive threads on consecutive outputs -----------
  for (int i = tid; i < d_out; i += LR_THREADS) {
    float acc[LR_SEQ];
#pragma unroll
    for (int s = 0; s < LR_SEQ; ++s) acc[s] = 0.f;
    for (int g = 0; g < G; ++g) {
      const float av = ptenc_to_float(Al[(size_t)i * G + g]);
#pragma unroll
      for (int s = 0; s < LR_SEQ; ++s) acc[s] = fmaf(av, w[s * G + g], acc[s]);
    }
#pragma unroll
    for (int s = 0; s < LR_SEQ; ++s) {
      if (s < nseq && (active == nullptr || active[b0 + s] != 0)) {
        T* dst = yl + (size_t)s * d_out + i;
        *dst = ptenc_from_float<T>(ptenc_to_float(*dst) + acc[s]);
      }
    }
  }
}

}  // namespace

cudaError_t ptenc_launch_lora_apply(ptenc_cache* c, int l0, int nl, const void* A, const void* Bm, const void* x,
                                    void* y, const uint8_t* active, int d_in, int d_out, cudaStream_t st) {
  const PtencDev& p = c->dev;
  const size_t smem = sizeof(float) * (size_t)LR_SEQ * (p.r + p.G);
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
