// Decode attention (step a2), shape-generic kernel: fp32 or bf16 storage, any head_dim <= 256 that is a
// multiple of 8, any query group size.  Sec. 3.1: o = softmax(q K^T / sqrt(d)) V over the live cache
// entries, the token appended last included.  Plain FFMA, fp32 throughout (no TF32), one CTA per
// (layer, sequence, query head); used for the fp32 configuration and for shapes the tensor-core kernel
// does not cover.
#include "ptenc_internal.h"

namespace {

constexpr int AG_THREADS = 128;
constexpr int AG_WARPS = AG_THREADS / 32;
constexpr int AG_MAXJ = 8;   // head_dim <= 32 * AG_MAXJ

template <typename T>
__global__ void __launch_bounds__(AG_THREADS)
k_attn_generic(PtencDev p, int l0, const T* __restrict__ q, const uint8_t* __restrict__ active,
               T* __restrict__ out, float* __restrict__ lse) {
  __shared__ float s_q[32 * AG_MAXJ];
  __shared__ float s_acc[AG_WARPS][32 * AG_MAXJ];
  __shared__ float s_m[AG_WARPS], s_l[AG_WARPS];

  const int D = p.D, W = p.W;
  int idx = blockIdx.x;
  const int hq = idx % p.Hq; idx /= p.Hq;
  const int b = idx % p.B;
  const int li = idx / p.B;
  const int l = l0 + li;
  if (active != nullptr && active[b] == 0) return;
  const size_t lb = (size_t)l * p.B + b;
  const int head = p.head[lb], count = p.count[lb];
  const int sink = p.n_sink != nullptr ? p.n_sink[lb] : 0;      // pinned prompt entries in slots [0, sink)
  const int cap = W - sink;
  if (count + sink <= 0) return;
  const int hkv = hq / p.g;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  const size_t qoff = (((size_t)li * p.B + b) * p.Hq + hq) * D;
  for (int d = tid; d < D; d += AG_THREADS) s_q[d] = ptenc_to_float(q[qoff + d]);
  __syncthreads();

  const T* Kb = reinterpret_cast<const T*>(p.K) + (lb * p.Hkv + hkv) * (size_t)W * D;
  const T* Vb = reinterpret_cast<const T*>(p.V) + (lb * p.Hkv + hkv) * (size_t)W * D;
  const float scale = 1.0f / sqrtf((float)D);

  float m = -INFINITY, lsum = 0.f;
  float acc[AG_MAXJ];
#pragma unroll
  for (int j = 0; j < AG_MAXJ; ++j) acc[j] = 0.f;

  for (int i = warp; i < sink + count; i += AG_WARPS) {
    int slot = i;
    if (i >= sink) {
      slot = head + (i - sink);
      if (slot >= cap) slot -= cap;
      slot += sink;
    }
    const T* kr = Kb + (size_t)slot * D;
    const T* vr = Vb + (size_t)slot * D;
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < AG_MAXJ; ++j) {
      const int d = lane + 32 * j;
      if (d < D) s = fmaf(s_q[d], ptenc_to_float(kr[d]), s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    s *= scale;
    const float m_new = fmaxf(m, s);
    const float corr = expf(m - m_new);       // exp(-inf) = 0 on the first token
    const float e = expf(s - m_new);
    lsum = lsum * corr + e;
#pragma unroll
    for (int j = 0; j < AG_MAXJ; ++j) {
      const int d = lane + 32 * j;
      if (d < D) acc[j] = acc[j] * corr + e * ptenc_to_float(vr[d]);
    }
    m = m_new;
  }
  if (lane == 0) { s_m[warp] = m; s_l[warp] = lsum; }
#pragma unroll
  for (int j = 0; j < AG_MAXJ; ++j) s_acc[warp][lane + 32 * j] = acc[j];
  __syncthreads();

  float mt = -INFINITY;
#pragma unroll
  for (int w = 0; w < AG_WARPS; ++w) mt = fmaxf(mt, s_m[w]);
  float lt = 0.f;
  float wgt[AG_WARPS];
#pragma unroll
  for (int w = 0; w < AG_WARPS; ++w) {
    wgt[w] = (s_m[w] == -INFINITY) ? 0.f : expf(s_m[w] - mt);
    lt += wgt[w] * s_l[w];
  }
  const float inv = 1.0f / lt;
  for (int d = tid; d < D; d += AG_THREADS) {
    float o = 0.f;
#pragma unroll
    for (int w = 0; w < AG_WARPS; ++w) o += wgt[w] * s_acc[w][d];
    out[qoff + d] = ptenc_from_float<T>(o * inv);
  }
  if (lse != nullptr && tid == 0) lse[((size_t)li * p.B + b) * p.Hq + hq] = mt + logf(lt);
}

}  // namespace

cudaError_t ptenc_launch_attn_generic(ptenc_cache* c, int l0, int nl, const void* q, const uint8_t* active,
                                      void* out, float* lse, cudaStream_t st) {
  const int grid = nl * c->cfg.batch * c->cfg.n_q_heads;
  if (c->cfg.dtype == PTENC_DTYPE_FP32)
    k_attn_generic<float><<<grid, AG_THREADS, 0, st>>>(c->dev, l0, (const float*)q, active, (float*)out, lse);
  else
    k_attn_generic<__nv_bfloat16><<<grid, AG_THREADS, 0, st>>>(c->dev, l0, (const __nv_bfloat16*)q, active,
                                                               (__nv_bfloat16*)out, lse);
  c->launches++;
  return cudaGetLastError();
}
