// Progressive encode of ONE evicted token per sequence (ring-per-step mode, E = 1) by a single warp.
//
// Sec. 3.3, Eq. (3) for m = 1: k_a = W^a_K k_e, v_a = W^a_V v_e, S' = (Q_a k_a) v_a^T, S <- Normalize(S + S').
// One warp folds one (layer, sequence): the evicted K and V rows (all KV heads concatenated) sit in the lanes'
// registers, the 2r dot products against the encoder weights stream the weights from L2 with 16-byte loads, and the
// rank-1 update of the [G, r] state runs a state row per lane.  Everything is fp32 except the stored rows and weights.
//
// The routine is the same wherever ring-per-step encoding happens -- on the spare warps of the attention kernel, where
// it overlaps the K/V stream of the same step, and in the stand-alone kernel behind ptenc_encode -- so the fused step
// and the separate calls give bit-identical states.
#pragma once

#include "ptenc_internal.h"

constexpr int ENCW_MAX_VEC = 4;        // 16-byte vectors of a row held per lane: d_kv <= 32 * 4 * 8 = 1024
constexpr int ENCW_MAX_RB = 4;         // 32-wide blocks of the rank: r <= 128
constexpr int ENCW_W_VEC = 8;          // 16-byte vectors of EACH weight matrix a lane keeps in flight: with NV vectors
                                       // per row and lane, 8 / NV output rows are requested per memory round trip

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

// NV = 16-byte vectors of a row per lane (2 or 4: d_kv <= 512, 1024).
template <int NV>
__device__ __forceinline__ void encw_fold_row_t(const PtencDev& p, int l, size_t lb, const __nv_bfloat16* rowK,
                                                const __nv_bfloat16* rowV, int lane) {
  constexpr int ENCW_JB = ENCW_W_VEC / NV;                   // 4 or 2 output rows per batch
  const int G = p.G, r = p.r, d_kv = p.d_kv;
  const int nv = d_kv >> 3;                                  // 16-byte vectors per row
  uint4 xk[NV], xv[NV];
#pragma unroll
  for (int u = 0; u < NV; ++u) {
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
  // The weights come from L2; a batch of ENCW_JB output rows is requested before any of it is used, so that a batch
  // costs one round trip, not one per row.
  float ka[ENCW_MAX_RB], va[ENCW_MAX_RB];
#pragma unroll
  for (int jb = 0; jb < ENCW_MAX_RB; ++jb) { ka[jb] = 0.f; va[jb] = 0.f; }
  for (int j0 = 0; j0 < r; j0 += ENCW_JB) {                  // r is a multiple of 8; a batch may run past r
    uint4 wk[ENCW_JB][NV], wv[ENCW_JB][NV];
#pragma unroll
    for (int jj = 0; jj < ENCW_JB; ++jj) {
#pragma unroll
      for (int u = 0; u < NV; ++u) {
        const int v = lane + 32 * u;
        if (v < nv && j0 + jj < r) {
          wk[jj][u] = __ldg(reinterpret_cast<const uint4*>(Wk + (size_t)(j0 + jj) * d_kv + (size_t)v * 8));
          wv[jj][u] = __ldg(reinterpret_cast<const uint4*>(Wv + (size_t)(j0 + jj) * d_kv + (size_t)v * 8));
        }
      }
    }
#pragma unroll
    for (int jj = 0; jj < ENCW_JB; ++jj) {
      if (j0 + jj >= r) break;                               // uniform over the warp
      float sk = 0.f, sv = 0.f;
#pragma unroll
      for (int u = 0; u < NV; ++u) {
        if (lane + 32 * u < nv) {
          sk += encw_dot8(wk[jj][u], xk[u]);
          sv += encw_dot8(wv[jj][u], xv[u]);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        sk += __shfl_xor_sync(0xffffffffu, sk, o);
        sv += __shfl_xor_sync(0xffffffffu, sv, o);
      }
      const int j = j0 + jj;
#pragma unroll
      for (int jb = 0; jb < ENCW_MAX_RB; ++jb)
        if ((j >> 5) == jb && lane == (j & 31)) { ka[jb] = sk; va[jb] = sv; }
    }
  }

  // ---- p = Q_a k_a; S <- Normalize(S + p v_a^T): a state row per lane -----------------------------------------------------
  // Rows are moved 32 values (eight 16-byte loads in flight) at a time.
  const float* Qa = p.Qa + (size_t)l * G * r;
  float* S = p.S + lb * (size_t)G * r;
  const bool row_mode = p.norm_mode == PTENC_NORM_ROW_L2;
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
        float4 qv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          qv[i] = (jb * 32 + 4 * i < r) ? *reinterpret_cast<const float4*>(qrow + jb * 32 + 4 * i)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i) {                        // lanes past r hold zeros in ka
          pg = fmaf(qv[i].x, __shfl_sync(0xffffffffu, ka[jb], 4 * i), pg);
          pg = fmaf(qv[i].y, __shfl_sync(0xffffffffu, ka[jb], 4 * i + 1), pg);
          pg = fmaf(qv[i].z, __shfl_sync(0xffffffffu, ka[jb], 4 * i + 2), pg);
          pg = fmaf(qv[i].w, __shfl_sync(0xffffffffu, ka[jb], 4 * i + 3), pg);
        }
      }
    }
    float ss = 0.f;
    const bool one_block = r <= 32;                          // the whole row fits the registers: scale before storing
#pragma unroll
    for (int jb = 0; jb < ENCW_MAX_RB; ++jb) {
      if (jb * 32 < r) {
        float4 sv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          sv[i] = (jb * 32 + 4 * i < r) ? *reinterpret_cast<const float4*>(srow + jb * 32 + 4 * i)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          sv[i].x = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], 4 * i), sv[i].x);
          sv[i].y = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], 4 * i + 1), sv[i].y);
          sv[i].z = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], 4 * i + 2), sv[i].z);
          sv[i].w = fmaf(pg, __shfl_sync(0xffffffffu, va[jb], 4 * i + 3), sv[i].w);
          ss = fmaf(sv[i].x, sv[i].x, ss);
          ss = fmaf(sv[i].y, sv[i].y, ss);
          ss = fmaf(sv[i].z, sv[i].z, ss);
          ss = fmaf(sv[i].w, sv[i].w, ss);
        }
        const float sc = (one_block && row_mode) ? rsqrtf(fmaxf(ss, 1e-24f)) : 1.f;      // 1 / max(|row|, 1e-12)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (valid && jb * 32 + 4 * i < r)
            *reinterpret_cast<float4*>(srow + jb * 32 + 4 * i) =
                make_float4(sv[i].x * sc, sv[i].y * sc, sv[i].z * sc, sv[i].w * sc);
        }
      }
    }
    if (valid) total += ss;
    if (row_mode && !one_block && valid) {                   // longer rows were stored un-normalised: rescale them
      const float sc = rsqrtf(fmaxf(ss, 1e-24f));
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

// rowK, rowV: the evicted token's key and value rows [d_kv] bf16 (16-byte aligned).  The whole warp must call.
__device__ __forceinline__ void encw_fold_row(const PtencDev& p, int l, size_t lb, const __nv_bfloat16* rowK,
                                              const __nv_bfloat16* rowV, int lane) {
  if (p.d_kv <= 512) encw_fold_row_t<2>(p, l, lb, rowK, rowV, lane);
  else encw_fold_row_t<4>(p, l, lb, rowK, rowV, lane);
}
