// Dynamic weight update (Sec. 3.3, Eq. (3)): Delta W = A S_e B, theta' = theta + Delta W, recomputed whenever the
// state changes.  Delta W is never formed: for the one token a sequence decodes per step,
//   y_b += Delta W_b x_b = A (S_b (B x_b)),
// three thin products per sequence (r x d_in, G x r, d_out x G).  Each sequence has its own state, so this is a
// batch of tiny products; the only sizeable traffic is A and B, which a CTA reads once for a block of sequences.
// fp32 accumulation throughout; x, y, A, B in the storage dtype.
#include <string.h>

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
    const int s = idx / G;
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

// ---------------------------------------------------------------------------------------------------------------
// bf16 path: three streaming kernels on warp-level mma, chained by programmatic dependent launch.  Sixteen sequences
// are the 16 rows of the A operand of mma.sync.m16n8k16.
//   k_lora_u   u = X B^T   a CTA per (layer, slice of d_in) keeps its column slice of B in shared memory and streams
//                          the inputs of every sequence of the layer through registers, a warp per 16 sequences;
//                          the slices' partial sums go to a scratch area [part][layer][sequence][r];
//   k_lora_w   w = S u     a warp per (layer, sequence): the partial sums are added in a fixed order, the state is
//                          read as one coalesced block, w leaves as two bf16 terms w_hi + w_lo so that nothing but
//                          the final rounding of y is lost;
//   k_lora_y   y += w A^T  a CTA per (layer, slice of d_out) keeps its rows of A in shared memory and streams the
//                          old outputs in and the new ones out, 16 bytes per lane and row.
// Every CTA of the two streaming kernels is resident at once (two per SM); the loads that do not depend on the kernel
// in front are requested before the wait for it.  (Folding the second product into the third kernel, the CTAs of a
// layer meeting at a counter, was slower: under load every dependent memory round trip costs about 2.5 us, and that
// version had more of them in a row.)
// One 16-byte load per lane feeds two mma steps: the contraction index is permuted the same way on both operands,
// which leaves the sums unchanged.
// ---------------------------------------------------------------------------------------------------------------
constexpr int LS_THREADS = 256;
constexpr int LS_WARPS = LS_THREADS / 32;
#ifndef PTENC_LORA_CTAS_PER_SM
#define PTENC_LORA_CTAS_PER_SM 2
#endif
constexpr int LS_SLOTS = 8;          // 32-wide chunks of the contraction / 32-wide groups of outputs a warp keeps in flight
constexpr int LS_SLOT_BYTES = LS_WARPS * LS_SLOTS * 2 * 32 * 16;   // per CTA: [warp][slot][row half][lane] 16 bytes

__device__ __forceinline__ void lr_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lr_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void ls_cp16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void ls_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void ls_cp_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
template <int N> __device__ __forceinline__ void ls_cp_wait_but() {      // all but the N most recent groups have landed
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ls_let_next_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void ls_wait_for_previous() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// bytes between the staged rows of B: the slice, padded so that the rows of a fragment load fall into distinct banks
__host__ __device__ inline int ls_b_stride(int np_max) { return (np_max * 64) | 64; }

// grid = (SL, nl).  u_part [SL * KS][nl][B][r] fp32.
template <int NT>                    // column tiles of u: r = 8 * NT
__global__ void __launch_bounds__(LS_THREADS, 2)
k_lora_u(PtencDev p, const __nv_bfloat16* __restrict__ Bm, const __nv_bfloat16* __restrict__ x,
         float* __restrict__ u_part, int d_in, int SL, int KS) {
  ls_let_next_start();
  extern __shared__ __align__(128) uint8_t ls_smem[];
  constexpr int r = 8 * NT;
  const int B = p.B, nl = gridDim.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qrow = lane >> 2, qcol = lane & 3;
  const int li = blockIdx.y, sl = blockIdx.x;
  const int n_pairs = d_in >> 5;
  const int p_lo = sl * n_pairs / SL, np = (sl + 1) * n_pairs / SL - p_lo;
  const int rs = ls_b_stride((n_pairs + SL - 1) / SL);
  const __nv_bfloat16* Bl = Bm + (size_t)li * r * d_in + (size_t)p_lo * 32;
  const __nv_bfloat16* xl = x + (size_t)li * B * d_in + (size_t)p_lo * 32;

  for (int row = warp; row < r; row += LS_WARPS)               // the slice of B: a warp per row, a lane per 16 bytes
    for (int v = lane; v < np * 4; v += 32) ls_cp16(ls_smem + (size_t)row * rs + v * 16, Bl + (size_t)row * d_in + v * 8);
  ls_cp_commit();

  // The streaming part is written as short rolled loops: a launch runs its code once, from instruction memory that
  // is in no cache, so every unrolled copy costs more than the loop overhead it saves.  A lane's 16-byte pieces
  // travel by asynchronous copy into shared-memory slots that only this lane reads (no barrier), LS_SLOTS chunks
  // ahead of the mma; one copy group is committed per chunk, empty past the end, so that "all but the LS_SLOTS - 1
  // most recent groups" always means "the chunk that is needed next".
  const int n_mt = (B + 15) >> 4;
  const int n_items = n_mt * KS;                               // (16 sequences, part of the slice) per warp pass
  uint4* slots = reinterpret_cast<uint4*>(ls_smem + (((size_t)r * rs + 127) & ~(size_t)127)) + warp * (LS_SLOTS * 2 * 32) + lane;
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  int item = warp;
  int c_lo = 0, c_hi = 0, b_lo = 0;
  const __nv_bfloat16* src_lo = xl;
  const __nv_bfloat16* src_hi = xl;
  auto open_item = [&]() {                                     // this warp's next item and its first LS_SLOTS chunks
    const int mt = item % n_mt, ks = item / n_mt;
    c_lo = ks * np / KS;
    c_hi = (ks + 1) * np / KS;
    b_lo = 16 * mt + qrow;
    src_lo = xl + (size_t)b_lo * d_in + qcol * 8;
    src_hi = src_lo + (size_t)8 * d_in;
  };
  auto request = [&](int c, int slot) {                        // chunk c of the item into a slot; one group either way
    if (c < c_hi) {
      if (b_lo < B) ls_cp16(slots + (2 * slot) * 32, src_lo + c * 32); else slots[(2 * slot) * 32] = zero;
      if (b_lo + 8 < B) ls_cp16(slots + (2 * slot + 1) * 32, src_hi + c * 32); else slots[(2 * slot + 1) * 32] = zero;
    }
    ls_cp_commit();
  };
  bool have = item < n_items;
  if (have) {
    open_item();
#pragma unroll 1
    for (int i = 0; i < LS_SLOTS; ++i) request(c_lo + i, i);
    ls_cp_wait_but<LS_SLOTS>();                                // the slice of B (the oldest group) has landed
  } else {
    ls_cp_wait_all();
  }
  __syncthreads();

  while (have) {
    float acc[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
#pragma unroll 1
    for (int c = c_lo; c < c_hi; ++c) {
      const int slot = (c - c_lo) % LS_SLOTS;
      ls_cp_wait_but<LS_SLOTS - 1>();
      const uint4 xa = slots[(2 * slot) * 32], xb = slots[(2 * slot + 1) * 32];
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        const uint4 bw = *reinterpret_cast<const uint4*>(ls_smem + (size_t)(t * 8 + qrow) * rs + c * 64 + qcol * 16);
        lr_mma(acc[t], xa.x, xb.x, xa.y, xb.y, bw.x, bw.y);
        lr_mma(acc[t], xa.z, xb.z, xa.w, xb.w, bw.z, bw.w);
      }
      request(c + LS_SLOTS, slot);
    }
    const int mt = item % n_mt, ks = item / n_mt;
    float* dst = u_part + (((size_t)(sl * KS + ks) * nl + li) * B + 16 * mt + qrow) * r + 2 * qcol;
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      if (b_lo < B) *reinterpret_cast<float2*>(dst + t * 8) = make_float2(acc[t][0], acc[t][1]);
      if (b_lo + 8 < B) *reinterpret_cast<float2*>(dst + (size_t)8 * r + t * 8) = make_float2(acc[t][2], acc[t][3]);
    }
    item += LS_WARPS;
    have = item < n_items;
    if (have) {
      open_item();
#pragma unroll 1
      for (int i = 0; i < LS_SLOTS; ++i) request(c_lo + i, i);
    }
  }
}

// grid = ceil(nl * B / 8) CTAs of 8 warps, a warp per (layer, sequence).  w_hi, w_lo [nl][B][G] bf16.
template <int LPR>                   // lanes that share a state row: r = 4 * LPR
__global__ void __launch_bounds__(LS_THREADS)
k_lora_w(PtencDev p, int l0, int nl, const float* __restrict__ u_part, int n_part, __nv_bfloat16* __restrict__ w_hi,
         __nv_bfloat16* __restrict__ w_lo) {
  ls_let_next_start();
  constexpr int r = 4 * LPR;
  constexpr int SB = 8;                                        // 16-byte vectors of the state requested together
  __shared__ __align__(16) float u_s[LS_WARPS][r];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int item = blockIdx.x * LS_WARPS + warp;
  const int B = p.B, G = p.G;
  const bool live = item < nl * B;
  const int li = live ? item / B : 0, b = live ? item - li * B : 0;
  const float4* Sv = reinterpret_cast<const float4*>(p.S + ((size_t)(l0 + li) * B + b) * G * r);
  const int n_vec = G * r / 4;                                 // a multiple of 32: G is a multiple of 32
  float4 sv[SB];
#pragma unroll
  for (int i = 0; i < SB; ++i)                                 // the state does not depend on the kernel in front
    sv[i] = (live && i * 32 + lane < n_vec) ? Sv[i * 32 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
  ls_wait_for_previous();
  if (live) {
    for (int j = lane; j < r; j += 32) {
      float v[PTENC_LORA_MAX_PART];                            // every part requested before the first is used
#pragma unroll
      for (int q = 0; q < PTENC_LORA_MAX_PART; ++q)
        v[q] = q < n_part ? u_part[(((size_t)q * nl + li) * B + b) * r + j] : 0.f;
      float t = 0.f;
#pragma unroll
      for (int q = 0; q < PTENC_LORA_MAX_PART; ++q) t += v[q];   // the same order in every launch
      u_s[warp][j] = t;
    }
  }
  __syncwarp();
  if (!live) return;
  const float4 uu = *reinterpret_cast<const float4*>(&u_s[warp][(lane % LPR) * 4]);
  for (int v0 = 0; v0 < n_vec; v0 += SB * 32) {
    if (v0 > 0) {
#pragma unroll
      for (int i = 0; i < SB; ++i)
        sv[i] = (v0 + i * 32 + lane < n_vec) ? Sv[v0 + i * 32 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int i = 0; i < SB; ++i) {
      float d = fmaf(sv[i].x, uu.x, fmaf(sv[i].y, uu.y, fmaf(sv[i].z, uu.z, sv[i].w * uu.w)));
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      const int vec = v0 + i * 32 + lane;
      if (vec < n_vec && (lane % LPR) == 0) {
        const int g = vec / LPR;
        const __nv_bfloat16 hi = __float2bfloat16_rn(d);
        w_hi[((size_t)li * B + b) * G + g] = hi;
        w_lo[((size_t)li * B + b) * G + g] = __float2bfloat16_rn(d - __bfloat162float(hi));
      }
    }
  }
}

// grid = (SO, nl).  Shared memory: the CTA's rows of A, one plane of 64-byte rows per 32 state rows, the four
// 16-byte pieces of a row permuted by (row / 8) % 4 so that a fragment load touches every bank once.
template <int KP>                    // G = 32 * KP
__global__ void __launch_bounds__(LS_THREADS, 2)
k_lora_y(PtencDev p, const __nv_bfloat16* __restrict__ A, __nv_bfloat16* __restrict__ y,
         const __nv_bfloat16* __restrict__ w_hi, const __nv_bfloat16* __restrict__ w_lo,
         const uint8_t* __restrict__ active, int d_out, int SO, int KS) {
  extern __shared__ __align__(128) uint8_t ls_smem[];
  constexpr int G = 32 * KP;
  const int B = p.B;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qrow = lane >> 2, qcol = lane & 3;
  const int li = blockIdx.y, so = blockIdx.x;
  const int n_groups = (d_out + 31) >> 5;                      // groups of 32 outputs
  const int g_lo = so * n_groups / SO, ng = (so + 1) * n_groups / SO - g_lo;
  const int plane = ((n_groups + SO - 1) / SO) * 32 * 64;      // bytes of a plane
  const __nv_bfloat16* Al = A + (size_t)li * d_out * G;
  __nv_bfloat16* yl = y + (size_t)li * B * d_out;

  for (int idx = tid; idx < ng * 32 * 4 * KP; idx += LS_THREADS) {
    const int o_rel = idx / (4 * KP), ch = idx - o_rel * 4 * KP;
    const int o = g_lo * 32 + o_rel;
    uint8_t* dst = ls_smem + (size_t)(ch >> 2) * plane + o_rel * 64 + (((ch & 3) ^ ((o_rel >> 3) & 3)) << 4);
    if (o < d_out) ls_cp16(dst, Al + (size_t)o * G + ch * 8);
    else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
  }
  ls_cp_commit();

  // rolled loops and lane-private slots as in k_lora_u: the old outputs of a group of 32 columns travel LS_SLOTS groups
  // ahead of the mma, one copy group per group of outputs
  const int n_mt = (B + 15) >> 4;
  const int n_items = n_mt * KS;                               // (16 sequences, part of the CTA's groups) per warp pass
  uint4* slots = reinterpret_cast<uint4*>(ls_smem + (size_t)KP * plane) + warp * (LS_SLOTS * 2 * 32) + lane;
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  int item = warp;
  int c_lo = 0, c_hi = 0, b_lo = 0;
  __nv_bfloat16* row_lo = yl;
  __nv_bfloat16* row_hi = yl;
  auto open_item = [&]() {
    const int mt = item % n_mt, ks = item / n_mt;
    c_lo = ks * ng / KS;
    c_hi = (ks + 1) * ng / KS;
    b_lo = 16 * mt + qrow;
    row_lo = yl + (size_t)b_lo * d_out + qcol * 8;
    row_hi = row_lo + (size_t)8 * d_out;
  };
  auto request = [&](int c, int slot) {                        // group c of the item's old outputs; one copy group either way
    const int o = (g_lo + c) * 32;
    if (c < c_hi && o + qcol * 8 < d_out) {
      if (b_lo < B) ls_cp16(slots + (2 * slot) * 32, row_lo + o); else slots[(2 * slot) * 32] = zero;
      if (b_lo + 8 < B) ls_cp16(slots + (2 * slot + 1) * 32, row_hi + o); else slots[(2 * slot + 1) * 32] = zero;
    }
    ls_cp_commit();
  };
  bool have = item < n_items;
  if (have) {
    open_item();
#pragma unroll 1
    for (int i = 0; i < LS_SLOTS; ++i) request(c_lo + i, i);   // in flight during the waits
  }
  ls_wait_for_previous();                                      // w is complete
  if (have) ls_cp_wait_but<LS_SLOTS>(); else ls_cp_wait_all(); // the rows of A (the oldest group) have landed
  __syncthreads();

  while (have) {
    const bool st_lo = b_lo < B && (active == nullptr || active[b_lo] != 0);
    const bool st_hi = b_lo + 8 < B && (active == nullptr || active[b_lo + 8] != 0);
    // the w fragments of the item's sixteen sequences
    uint4 wh_l[KP], wh_h[KP], wl_l[KP], wl_h[KP];
#pragma unroll
    for (int k = 0; k < KP; ++k) {
      const size_t o_lo = ((size_t)li * B + b_lo) * G + k * 32 + qcol * 8, o_hi = o_lo + (size_t)8 * G;
      wh_l[k] = b_lo < B ? *reinterpret_cast<const uint4*>(w_hi + o_lo) : zero;
      wl_l[k] = b_lo < B ? *reinterpret_cast<const uint4*>(w_lo + o_lo) : zero;
      wh_h[k] = b_lo + 8 < B ? *reinterpret_cast<const uint4*>(w_hi + o_hi) : zero;
      wl_h[k] = b_lo + 8 < B ? *reinterpret_cast<const uint4*>(w_lo + o_hi) : zero;
    }
#pragma unroll 1
    for (int c = c_lo; c < c_hi; ++c) {
      const int slot = (c - c_lo) % LS_SLOTS;
      ls_cp_wait_but<LS_SLOTS - 1>();
      const uint4 old_lo = slots[(2 * slot) * 32], old_hi = slots[(2 * slot + 1) * 32];
      const int o = (g_lo + c) * 32 + qcol * 8;
      float acc[4][4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
        // column n of tile t is output 8 * (n / 2) + 2 * t + (n % 2) of the group: this lane's columns of the four
        // tiles are eight consecutive outputs
        const int o_rel = c * 32 + 8 * (qrow >> 1) + 2 * t + (qrow & 1);
#pragma unroll
        for (int k = 0; k < KP; ++k) {
          const uint4 aw = *reinterpret_cast<const uint4*>(ls_smem + (size_t)k * plane + o_rel * 64 +
                                                           ((qcol ^ ((o_rel >> 3) & 3)) << 4));
          lr_mma(acc[t], wh_l[k].x, wh_h[k].x, wh_l[k].y, wh_h[k].y, aw.x, aw.y);
          lr_mma(acc[t], wh_l[k].z, wh_h[k].z, wh_l[k].w, wh_h[k].w, aw.z, aw.w);
          lr_mma(acc[t], wl_l[k].x, wl_h[k].x, wl_l[k].y, wl_h[k].y, aw.x, aw.y);
          lr_mma(acc[t], wl_l[k].z, wl_h[k].z, wl_l[k].w, wl_h[k].w, aw.z, aw.w);
        }
      }
      if (o < d_out) {
        const uint32_t ol[4] = {old_lo.x, old_lo.y, old_lo.z, old_lo.w}, oh[4] = {old_hi.x, old_hi.y, old_hi.z, old_hi.w};
        uint32_t nlo[4], nhi[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const __nv_bfloat162 va = *reinterpret_cast<const __nv_bfloat162*>(&ol[t]);
          const __nv_bfloat162 vb = *reinterpret_cast<const __nv_bfloat162*>(&oh[t]);
          nlo[t] = lr_pack(__low2float(va) + acc[t][0], __high2float(va) + acc[t][1]);
          nhi[t] = lr_pack(__low2float(vb) + acc[t][2], __high2float(vb) + acc[t][3]);
        }
        if (st_lo) *reinterpret_cast<uint4*>(row_lo + (g_lo + c) * 32) = make_uint4(nlo[0], nlo[1], nlo[2], nlo[3]);
        if (st_hi) *reinterpret_cast<uint4*>(row_hi + (g_lo + c) * 32) = make_uint4(nhi[0], nhi[1], nhi[2], nhi[3]);
      }
      request(c + LS_SLOTS, slot);
    }
    item += LS_WARPS;
    have = item < n_items;
    if (have) {
      open_item();
#pragma unroll 1
      for (int i = 0; i < LS_SLOTS; ++i) request(c_lo + i, i);
    }
  }
}

template <typename... KArgs, typename... Args>
cudaError_t ls_launch(void (*kernel)(KArgs...), dim3 grid, size_t smem, bool after_previous, cudaStream_t st,
                      Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = dim3(LS_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (after_previous) {
    // programmatic dependent launch: the grid may become resident while the kernel in front of it on the stream
    // (which signals that it allows this) is still running; the kernel waits before it reads that kernel's results
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

constexpr size_t LS_SMEM_MAX = 112 * 1024;  // per CTA, so that two CTAs fit an SM

// The streaming path: bf16, r in {16, 32, 64}, G in {32, 64, 96, 128}, d_in a multiple of 32, d_out a multiple of 8.
cudaError_t ls_apply(ptenc_cache* c, int l0, int nl, const __nv_bfloat16* A, const __nv_bfloat16* Bm,
                     const __nv_bfloat16* x, __nv_bfloat16* y, const uint8_t* active, int d_in, int d_out,
                     cudaStream_t st, bool* taken) {
  const PtencDev& p = c->dev;
  *taken = false;
  if (c->cfg.dtype != PTENC_DTYPE_BF16 || (p.r != 16 && p.r != 32 && p.r != 64) || (p.G & 31) != 0 || p.G > 128 ||
      (d_in & 31) != 0 || (d_out & 7) != 0 || nl > 65535)
    return cudaSuccess;
  static bool attr_done[PTENC_MAX_DEVICES] = {};
  if (ptenc_first_use(attr_done, c->cfg.device)) {
    cudaError_t e = cudaSuccess;
    auto big = [&](const void* f) {
      if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LS_SMEM_MAX);
    };
    big((const void*)k_lora_u<2>); big((const void*)k_lora_u<4>); big((const void*)k_lora_u<8>);
    big((const void*)k_lora_y<1>); big((const void*)k_lora_y<2>); big((const void*)k_lora_y<3>); big((const void*)k_lora_y<4>);
    if (e != cudaSuccess) return e;
  }
  const int n_mt = (p.B + 15) / 16;
  const int want = PTENC_LORA_CTAS_PER_SM * c->sm_count;        // CTAs of a streaming kernel: all resident at once
  // slices of d_in: enough CTAs, a slice of B that fits shared memory, no more partial sums than the scratch holds
  const int n_pairs = d_in >> 5;
  int SL = want / nl;                                           // never a second, nearly empty wave
  if (SL < 1) SL = 1;
  if (SL > n_pairs) SL = n_pairs;
  if (SL > PTENC_LORA_MAX_PART) SL = PTENC_LORA_MAX_PART;
  while (SL < n_pairs && (size_t)p.r * ls_b_stride((n_pairs + SL - 1) / SL) + 128 + LS_SLOT_BYTES > LS_SMEM_MAX) ++SL;
  if (SL > PTENC_LORA_MAX_PART) return cudaSuccess;
  int KS = LS_WARPS / n_mt;                                     // idle warps take parts of the slice
  if (KS < 1) KS = 1;
  if (SL * KS > PTENC_LORA_MAX_PART) KS = PTENC_LORA_MAX_PART / SL;
  const size_t smem_u = (((size_t)p.r * ls_b_stride((n_pairs + SL - 1) / SL) + 127) & ~(size_t)127) + LS_SLOT_BYTES;
  if (smem_u > LS_SMEM_MAX) return cudaSuccess;
  // slices of d_out
  const int n_groups = (d_out + 31) >> 5;
  const int KP = p.G >> 5;
  int SO = want / nl;
  if (SO < 1) SO = 1;
  if (SO > n_groups) SO = n_groups;
  while (SO < n_groups && (size_t)KP * ((n_groups + SO - 1) / SO) * 32 * 64 + LS_SLOT_BYTES > LS_SMEM_MAX) ++SO;
  const size_t smem_y = (size_t)KP * ((n_groups + SO - 1) / SO) * 32 * 64 + LS_SLOT_BYTES;
  if (smem_y > LS_SMEM_MAX) return cudaSuccess;
  int KS2 = LS_WARPS / n_mt;
  if (KS2 < 1) KS2 = 1;
  *taken = true;
  __nv_bfloat16* w_hi = c->lora_w;
  __nv_bfloat16* w_lo = c->lora_w + (size_t)p.L * p.B * p.G;
  const float* u_c = c->lora_u;
  cudaError_t e;
  switch (p.r) {
    case 16: e = ls_launch(k_lora_u<2>, dim3(SL, nl), smem_u, false, st, p, Bm, x, c->lora_u, d_in, SL, KS); break;
    case 32: e = ls_launch(k_lora_u<4>, dim3(SL, nl), smem_u, false, st, p, Bm, x, c->lora_u, d_in, SL, KS); break;
    default: e = ls_launch(k_lora_u<8>, dim3(SL, nl), smem_u, false, st, p, Bm, x, c->lora_u, d_in, SL, KS); break;
  }
  c->launches++;
  if (e != cudaSuccess) return e;
  const dim3 gw((nl * p.B + LS_WARPS - 1) / LS_WARPS);
  switch (p.r) {
    case 16: e = ls_launch(k_lora_w<4>, gw, 0, true, st, p, l0, nl, u_c, SL * KS, w_hi, w_lo); break;
    case 32: e = ls_launch(k_lora_w<8>, gw, 0, true, st, p, l0, nl, u_c, SL * KS, w_hi, w_lo); break;
    default: e = ls_launch(k_lora_w<16>, gw, 0, true, st, p, l0, nl, u_c, SL * KS, w_hi, w_lo); break;
  }
  c->launches++;
  if (e != cudaSuccess) return e;
  const __nv_bfloat16* w_hi_c = w_hi;
  const __nv_bfloat16* w_lo_c = w_lo;
  switch (KP) {
    case 1: e = ls_launch(k_lora_y<1>, dim3(SO, nl), smem_y, true, st, p, A, y, w_hi_c, w_lo_c, active, d_out, SO, KS2); break;
    case 2: e = ls_launch(k_lora_y<2>, dim3(SO, nl), smem_y, true, st, p, A, y, w_hi_c, w_lo_c, active, d_out, SO, KS2); break;
    case 3: e = ls_launch(k_lora_y<3>, dim3(SO, nl), smem_y, true, st, p, A, y, w_hi_c, w_lo_c, active, d_out, SO, KS2); break;
    default: e = ls_launch(k_lora_y<4>, dim3(SO, nl), smem_y, true, st, p, A, y, w_hi_c, w_lo_c, active, d_out, SO, KS2); break;
  }
  c->launches++;
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t ptenc_launch_lora_apply(ptenc_cache* c, int l0, int nl, const void* A, const void* Bm, const void* x,
                                    void* y, const uint8_t* active, int d_in, int d_out, cudaStream_t st) {
  const PtencDev& p = c->dev;
  {
    bool taken = false;
    cudaError_t e = ls_apply(c, l0, nl, (const __nv_bfloat16*)A, (const __nv_bfloat16*)Bm, (const __nv_bfloat16*)x,
                             (__nv_bfloat16*)y, active, d_in, d_out, st, &taken);
    if (taken || e != cudaSuccess) return e;
  }
  const size_t smem = sizeof(float) * ((((size_t)LR_SEQ * (p.r + p.G) + 3) & ~(size_t)3) +
                                       (((size_t)LR_SEQ * p.G * (p.r + 1) + 3) & ~(size_t)3)) +
                      (size_t)LR_SEQ * d_in * p.elt;
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  static bool attr_done[PTENC_MAX_DEVICES] = {};
  if (ptenc_first_use(attr_done, c->cfg.device)) {
    cudaError_t e = cudaFuncSetAttribute(k_lora_apply<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_lora_apply<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
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
