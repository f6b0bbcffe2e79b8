// Progressive encode of ONE evicted token per sequence (ring-per-step mode, E = 1) by a single warp.
//
// Sec. 3.3, Eq. (3) for m = 1: k_a = W^a_K k_e, v_a = W^a_V v_e, S' = (Q_a k_a) v_a^T, S <- Normalize(S + S').
// One warp folds one (layer, sequence): the evicted K and V rows (all KV heads concatenated) sit in the lanes'
// registers, the 2r dot products against the encoder weights stream the weights from L2 with 16-byte loads, and the
// rank-1 update of the [G, r] state runs a state row per lane.  Everything is fp32 except the stored rows and weights.
//
// The routine is the same wherever ring-per-step encoding happens -- in the spare warp of the attention kernel, where
// it overlaps the K/V stream of the same step, and in the stand-alone kernel behind ptenc_encode -- so the fused step
// and the separate calls give bit-identical states.
#pragma once

#include "ptenc_internal.h"

constexpr int ENCW_MAX_VEC = 4;        // 16-byte vectors of a row held per lane: d_kv <= 32 * 4 * 8 = 1024
constexpr int ENCW_MAX_RB = 4;         // 32-wide blocks of the rank: r <= 128

__device__ __forceinline__ float encw_dot8(const uint4& w, const uint4& x) {
  const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&w);
  const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&x);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 a = __bfloat1622float2(wp[i]), b = __bfloat1622float2(xp[i]);
    s = fmaf(a.x, b.x, s);
    s = fmaf(a.y, b.y, s);
  }
  return s;
}

// Shapes this routine covers (bf16 storage is checked by the caller).
__host__ __device__ inline bool encw_shape_ok(int G, int r, int d_kv) {
  return (r & 7) == 0 && r <= 32 * ENCW_MAX_RB && (d_kv & 31) == 0 && d_kv <= 256 * ENCW_MAX_VEC && G >= 1 && G <= 128;
}

// rowK, rowV: the evicted token's key and value rows [d_kv] bf16 (16-byte aligned).  The whole warp must call.
__device__ __forceinline__ void encw_fold_row(const PtencDev& p, int l, size_t lb, const __nv_bfloat16* rowK,
                                              const __nv_bfloat16* rowV, int lane) {
  const int G = p.G, r = p.r, d_kv = p.d_kv;
  const int nv = d_kv >> 3;                                  // 16-byte vectors per row
  uint4 xk[ENCW_MAX_VEC], xv[ENCW_MAX_VEC];
#pragma unroll
  for (int u = 0; u < ENCW_MAX_VEC; ++u) {
    const int v = lane + 32 * u;
    xk[u] = make_uint4(0u, 0u, 0u, 0u);
    xv[u] = xk[u];
    if (v < nv) {
      xk[u] = *reinterpret_cast<const uint4*>(rowK + (size_t)v * 8);
      xv[u] = *reinterpret_cast<const uint4*>(rowV + (size_t)v * 8);
    }
  }
  const __nv_bfloat16* Wk = reinterpret_cast<const __nv_bfloat16*>(p.Wk) + (size_t)l * r * d_kv;
  const __nv_bfloat16* Wv = reinterpret_cast<const __nv_bfloat16*>(p.Wv) + (size_t)l * r * d_kv;

  // ---- k_a = W^a_K k_e, v_a = W^a_V v_e: element j ends up in lane j % 32, register j / 32 ------------------------------
  float ka[ENCW_MAX_RB], va[ENCW_MAX_RB];
#pragma unroll
  for (int jb = 0; jb < ENCW_MAX_RB; ++jb) {
    ka[jb] = 0.f;
    va[jb] = 0.f;
    if (jb * 32 < r) {
#pragma unroll 4
      for (int jj = 0; jj < 32; ++jj) {
        const int j = jb * 32 + jj;
        if (j < r) {                                         // uniform over the warp
          float sk = 0.f, sv = 0.f;
#pragma unroll
          for (int u = 0; u < ENCW_MAX_VEC; ++u) {
            const int v = lane + 32 * u;
            if (v < nv) {
              const uint4 wk = __ldg(reinterpret_cast<const uint4*>(Wk + (size_t)j * d_kv + (size_t)v * 8));
              const uint4 wv = __ldg(reinterpret_cast<const uint4*>(Wv + (size_t)j * d_kv + (size_t)v * 8));
              sk += encw_dot8(wk, xk[u]);
              sv += encw_dot8(wv, xv[u]);
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            sk += __shfl_xor_sync(0xffffffffu, sk, o);
            sv += __shfl_xor_sync(0xffffffffu, sv, o);
          }
          if (lane == jj) { ka[jb] = sk; va[jb] = sv; }
        }
      }
    }
  }

  // ---- p = Q_a k_a; S <- Normalize(S + p v_a^T): a state row per lane -----------------------------------------------------
  const float* Qa = p.Qa + (size_t)l * G * r;
  float* S = p.S + lb * (size_t)G * r;
  float total = 0.f;
  for (int g0 = 0; g0 < G; g0 += 32) {
    const int g = g0 + lane;
    const bool valid = g < G;
    const float* qrow = Qa + (size_t)(valid ? g : 0) * r;
    float* srow = S + (size_t)(valid ? g : 0) * r;
    float pg = 0.f;
#pragma unroll
    for (int jb = 0; jb < ENCW_MAX_RB; ++jb) {
      if (jb * 32 < r) {
        for (int jj = 0; jj < 32 && jb * 32 + jj < r; jj += 4) {
          const float4 qv = *reinterpret_cast<const float4*>(qrow + jb * 32 + jj);
          pg = fmaf(qv.x, __shfl_sync(0xffffffffu, ka[jb], jj), pg);
          pg = fmaf(qv.y, __shfl_sync(0xffffffffu, ka[jb], jj + 1), pg);
          pg = fmaf(qv.z, __shfl_sync(0xffffffffu, ka[jb], jj + 2), pg);
          pg = fmaf(qv.w, __shfl_sync(0xffffffffu, ka[jb], jj + 3), pg);
        }
      }
    }
    float ss = 0.f;
#pragma unroll
    for (int jb = 0; jb < ENCW_MAX_RB; ++jb) {
      if (jb * 32 < r) {
        for (int jj = 0; jj < 32 && jb * 32 + jj < r; jj += 4) {
          float4 sv = *reinterpret_cast<const float4*>(srow + jb * 32 + jj);
          sv.x = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], jj), sv.x);
          sv.y = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], jj + 1), sv.y);
          sv.z = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], jj + 2), sv.z);
          sv.w = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], jj + 3), sv.w);
          ss = fmaf(sv.x, sv.x, ss);
          ss = fmaf(sv.y, sv.y, ss);
          ss = fmaf(sv.z, sv.z, ss);
          ss = fmaf(sv.w, sv.w, ss);
          if (valid) *reinterpret_cast<float4*>(srow + jb * 32 + jj) = sv;       // the un-normalised sum
        }
      }
    }
    if (valid) total += ss;
    if (p.norm_mode == PTENC_NORM_ROW_L2 && valid) {
      const float sc = rsqrtf(fmaxf(ss, 1e-24f));            // 1 / max(|row|, 1e-12)
      for (int j = 0; j < r; j += 4) {
        float4 sv = *reinterpret_cast<const float4*>(srow + j);
        sv.x *= sc; sv.y *= sc; sv.z *= sc; sv.w *= sc;
        *reinterpret_cast<float4*>(srow + j) = sv;
      }
    }
  }
  if (p.norm_mode == PTENC_NORM_FROBENIUS) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    const float sc = 1.f / fmaxf(sqrtf(total), 1e-12f);
    for (int g = lane; g < G; g += 32) {                     // each lane rescales the rows it wrote itself
      float* srow = S + (size_t)g * r;
      for (int j = 0; j < r; j += 4) {
        float4 sv = *reinterpret_cast<const float4*>(srow + j);
        sv.x *= sc; sv.y *= sc; sv.z *= sc; sv.w *= sc;
        *reinterpret_cast<float4*>(srow + j) = sv;
      }
    }
  }
}
