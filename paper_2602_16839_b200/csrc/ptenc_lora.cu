// Dynamic weight update (Sec. 3.3, Eq. (3)): Delta W = A S_e B, theta' = theta + Delta W, recomputed whenever the
// state changes.  Delta W is never formed: for the one token a sequence decodes per step,
//   y_b += Delta W_b x_b = A (S_b (B x_b)),
// three thin products per sequence (r x d_in, G x r, d_out x G).  Each sequence has its own state, so this is a
// batch of tiny products; the only sizeable traffic is A and B, which a CTA reads once for a block of sequences.
// fp32 accumulation throughout; x, y, A, B in the storage dtype.
#include <cooperative_groups.h>

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
// bf16 path: warp-level mma inside a thread-block cluster.  Sixteen sequences are the 16 rows of the A operand; the
// four CTAs of a cluster share one (layer, block of 16 sequences):
//   phase 1  u = X B^T     each CTA contracts its quarter of d_in (A fragments straight from the inputs, B fragments
//                          straight from B, both with one 16-byte load per lane feeding two mma steps; the contraction
//                          index is permuted the same way on both operands, which leaves the sums unchanged); the
//                          partial sums meet through distributed shared memory;
//   phase 2  w = S u       fp32, each CTA for four of the sixteen sequences, a lane per state row; w is split into two
//                          bf16 terms w_hi + w_lo so that nothing but the final rounding of y is lost; the quarters are
//                          gathered through distributed shared memory;
//   phase 3  y += w A^T    each CTA for its quarter of d_out, A's rows as the B operand.
// Splitting a block four ways makes the call 4 x as many, smaller CTAs: all of them are resident at once (one wave),
// every weight byte is still read once per 16 sequences, and the three dependent phases of one block overlap with
// those of the others on the same SM.
// ---------------------------------------------------------------------------------------------------------------
constexpr int LM_SEQ = 16;
constexpr int LM_CLUSTER = 4;
constexpr int LM_THREADS = 256;
constexpr int LM_WARPS = LM_THREADS / 32;

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
__host__ __device__ inline int lm_k_split(int r) {
  const int tiles = r >> 3;
  return tiles < LM_WARPS ? LM_WARPS / tiles : 1;
}
// Shared memory of a CTA: a staging buffer (first the CTA's column slice of the 16 input rows and of B's r rows,
// later its slice of A's rows), then u partials [KS][16][r] fp32, u of this CTA [16][r] fp32, w_hi and w_lo [16][G] bf16.
__host__ __device__ inline int lm_slice_pairs(int d_in) { return ((d_in >> 5) + LM_CLUSTER - 1) / LM_CLUSTER; }
__host__ __device__ inline int lm_row_stride(int d_in) { return lm_slice_pairs(d_in) * 64 + 64; }   // bytes; 64 mod 128
__host__ __device__ inline int lm_slice_tiles(int d_out) { return ((d_out >> 3) + LM_CLUSTER - 1) / LM_CLUSTER; }
__host__ __device__ inline size_t lm_a_bytes(int G, int d_out) {          // the CTA's rows of A, 128-byte aligned
  return (((size_t)lm_slice_tiles(d_out) * 8 * G * 2) + 127) & ~(size_t)127;
}
__host__ __device__ inline int lm_y_stride(int d_out) { return lm_slice_tiles(d_out) * 16 + 16; }    // bytes
__host__ __device__ inline size_t lm_stage_bytes(int G, int r, int d_in, int d_out) {
  const size_t in_bytes = (size_t)(LM_SEQ + r) * lm_row_stride(d_in);
  const size_t a_bytes = lm_a_bytes(G, d_out) + (size_t)LM_SEQ * lm_y_stride(d_out);
  return ((in_bytes > a_bytes ? in_bytes : a_bytes) + 127) & ~(size_t)127;
}
__host__ __device__ inline size_t lr_mma_smem(int G, int r, int d_in, int d_out) {
  return lm_stage_bytes(G, r, d_in, d_out) + (size_t)(lm_k_split(r) + 1) * LM_SEQ * r * 4 + (size_t)2 * LM_SEQ * G * 2;
}

__device__ __forceinline__ void lm_cp16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void lm_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void lm_cp_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// grid = (LM_CLUSTER, nl * ceil(B / 16)), cluster = (LM_CLUSTER, 1, 1).
// Every global read of a CTA is requested up front or as early as its buffer is free, so that a CTA pays about two
// memory round trips in all: the column slices of the inputs and of B go to shared memory with asynchronous copies,
// the state rows and the old outputs go to registers, and the CTA's rows of A follow into the same buffer as soon as
// the first product is done (while the partial sums travel through the cluster).
__global__ void __cluster_dims__(LM_CLUSTER, 1, 1) __launch_bounds__(LM_THREADS, 2)
k_lora_apply_cluster(PtencDev p, int l0, const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ Bm,
                     const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y,
                     const uint8_t* __restrict__ active, int d_in, int d_out) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(128) uint8_t lm_smem[];
  const int G = p.G, r = p.r, B = p.B;
  const int n_tiles = r >> 3;                                   // column tiles of u
  const int KS = lm_k_split(r);                                 // warps sharing a tile split the CTA's slice of d_in
  uint8_t* stage = lm_smem;
  float* u_part = reinterpret_cast<float*>(lm_smem + lm_stage_bytes(G, r, d_in, d_out));   // [KS][16][r]
  float* u_loc = u_part + KS * LM_SEQ * r;                      // [16][r] this CTA's share of the contraction
  __nv_bfloat16* w_hi = reinterpret_cast<__nv_bfloat16*>(u_loc + LM_SEQ * r);    // [16][G]
  __nv_bfloat16* w_lo = w_hi + LM_SEQ * G;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qrow = lane >> 2, qcol = lane & 3;
  const int rank = (int)cluster.block_rank();                   // = blockIdx.x
  const int nblk = (B + LM_SEQ - 1) / LM_SEQ;
  const int li = blockIdx.y / nblk;
  const int b0 = (blockIdx.y - li * nblk) * LM_SEQ;
  const int l = l0 + li;
  const int nseq = min(LM_SEQ, B - b0);
  const __nv_bfloat16* Bl = Bm + (size_t)li * r * d_in;
  const __nv_bfloat16* Al = A + (size_t)li * d_out * G;
  const __nv_bfloat16* xl = x + ((size_t)li * B + b0) * d_in;
  __nv_bfloat16* yl = y + ((size_t)li * B + b0) * d_out;
  const bool lo_ok = qrow < nseq, hi_ok = qrow + 8 < nseq;      // the two sequences whose rows this lane touches

  // this CTA's shares: pairs of mma steps along d_in, tiles of 8 outputs along d_out, sequences of the block
  const int n_pairs = d_in >> 5;
  const int p_lo = rank * n_pairs / LM_CLUSTER, p_hi = (rank + 1) * n_pairs / LM_CLUSTER;
  const int np = p_hi - p_lo;
  const int n_out_tiles = d_out >> 3;
  const int t_lo = rank * n_out_tiles / LM_CLUSTER, t_hi = (rank + 1) * n_out_tiles / LM_CLUSTER;
  const int s_first = rank * (LM_SEQ / LM_CLUSTER);
  const int rs = lm_row_stride(d_in);                           // bytes between staged rows

  // ---- requests: input and B column slices -> shared memory (rows 0..15 inputs, 16.. B) ---------------------------------
  {
    const int vec_per_row = np * 4;                             // 16-byte vectors of a row's slice
    const int rows = LM_SEQ + r;
    for (int row = warp; row < rows; row += LM_WARPS) {         // a warp per row, a lane per 16 bytes
      uint8_t* drow = stage + (size_t)row * rs;
      const __nv_bfloat16* srow = row < LM_SEQ ? xl + (size_t)row * d_in + (size_t)p_lo * 32
                                               : Bl + (size_t)(row - LM_SEQ) * d_in + (size_t)p_lo * 32;
      const bool real = row >= LM_SEQ || row < nseq;
      for (int v = lane; v < vec_per_row; v += 32) {
        if (real) lm_cp16(drow + v * 16, srow + v * 8);
        else *reinterpret_cast<uint4*>(drow + v * 16) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    lm_cp_commit();
  }
  // ---- requests: the state rows this thread needs in phase 2 (a warp per sequence, a lane per state row; r <= 32 * 4) -----
  // and the old outputs of this lane's positions in the CTA's output tiles (phase 3) -> registers
  const int sq = warp;                                          // sequence of this CTA's four handled by this warp
  const bool s_warp = sq < LM_SEQ / LM_CLUSTER && s_first + sq < nseq;
  lm_cp_wait_all();
  __syncthreads();

  // ---- phase 1: u (this CTA's slice of d_in), fragments from shared memory ------------------------------------------------
  {
    for (int item = warp; item < n_tiles * KS; item += LM_WARPS) {
      const int tile = item % n_tiles, ks = item / n_tiles;
      const int s_lo = ks * np / KS, s_hi = (ks + 1) * np / KS;
      const uint8_t* wrow = stage + (size_t)(LM_SEQ + tile * 8 + qrow) * rs + qcol * 16;
      const uint8_t* xlo = stage + (size_t)qrow * rs + qcol * 16;
      const uint8_t* xhi = xlo + (size_t)8 * rs;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
      for (int s0 = s_lo; s0 < s_hi; ++s0) {
        const uint4 bw = *reinterpret_cast<const uint4*>(wrow + s0 * 64);
        const uint4 al = *reinterpret_cast<const uint4*>(xlo + s0 * 64);
        const uint4 ah = *reinterpret_cast<const uint4*>(xhi + s0 * 64);
        lr_mma(c, al.x, ah.x, al.y, ah.y, bw.x, bw.y);
        lr_mma(c, al.z, ah.z, al.w, ah.w, bw.z, bw.w);
      }
      float* dst = u_part + ((size_t)ks * LM_SEQ + qrow) * r + tile * 8 + 2 * qcol;
      dst[0] = c[0];
      dst[1] = c[1];
      dst[8 * r] = c[2];
      dst[8 * r + 1] = c[3];
    }
  }
  __syncthreads();
  // the staging buffer is free: this CTA's rows of A follow into it while the partial sums are exchanged
  uint8_t* ystage = stage + lm_a_bytes(G, d_out);               // [16][ys] the block's old outputs, this CTA's columns
  const int ys = lm_y_stride(d_out);
  {
    const size_t bytes = (size_t)(t_hi - t_lo) * 8 * G * 2;
    const char* src = reinterpret_cast<const char*>(Al + (size_t)t_lo * 8 * G);
    for (size_t o = (size_t)tid * 16; o < bytes; o += (size_t)LM_THREADS * 16) lm_cp16(stage + o, src + o);
    const int yv = t_hi - t_lo;                                 // 16-byte vectors (one output tile) per row
    for (int row = warp; row < nseq; row += LM_WARPS)
      for (int v = lane; v < yv; v += 32)
        lm_cp16(ystage + (size_t)row * ys + v * 16, yl + (size_t)row * d_out + (size_t)(t_lo + v) * 8);
    lm_cp_commit();
  }
  for (int i = tid; i < LM_SEQ * r; i += LM_THREADS) {
    float t = u_part[i];
    for (int ks = 1; ks < KS; ++ks) t += u_part[(size_t)ks * LM_SEQ * r + i];
    u_loc[i] = t;
  }
  cluster.sync();                                              // every CTA's share of u is in its shared memory

  // ---- phase 2: w = S u for this CTA's four sequences (a warp per sequence, a lane per state row) -----------------------
  {
    const float* u_rem[LM_CLUSTER];
#pragma unroll
    for (int c = 0; c < LM_CLUSTER; ++c) u_rem[c] = cluster.map_shared_rank(u_loc, c);
    if (sq < LM_SEQ / LM_CLUSTER) {
      const int s = s_first + sq;
      for (int g = lane; g < G; g += 32) {
        float acc = 0.f;
        if (s_warp) {
          const float* Srow = p.S + (((size_t)l * B + b0 + s) * G + g) * r;
          for (int j0 = 0; j0 < r; j0 += 32) {                  // eight 16-byte loads of the state row in flight
            float4 sv[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
              sv[i] = (j0 + 4 * i < r) ? *reinterpret_cast<const float4*>(Srow + j0 + 4 * i)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int j = j0 + 4 * i;
              if (j < r) {
                float4 uu = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int c = 0; c < LM_CLUSTER; ++c) {           // the same order in every CTA
                  const float4 t = *reinterpret_cast<const float4*>(u_rem[c] + (size_t)s * r + j);
                  uu.x += t.x; uu.y += t.y; uu.z += t.z; uu.w += t.w;
                }
                acc = fmaf(sv[i].x, uu.x, acc);
                acc = fmaf(sv[i].y, uu.y, acc);
                acc = fmaf(sv[i].z, uu.z, acc);
                acc = fmaf(sv[i].w, uu.w, acc);
              }
            }
          }
        }
        const __nv_bfloat16 hi = __float2bfloat16_rn(acc);
        w_hi[s * G + g] = hi;
        w_lo[s * G + g] = __float2bfloat16_rn(acc - __bfloat162float(hi));
      }
    }
  }
  cluster.sync();                                              // every CTA's four rows of w are in its shared memory
  // gather the other CTAs' rows of w (16 x G bf16 twice: a few KB)
  {
    const int per_cta = (LM_SEQ / LM_CLUSTER) * G;               // elements of w_hi (and of w_lo) a CTA produced
    for (int c = 0; c < LM_CLUSTER; ++c) {
      if (c == rank) continue;
      const __nv_bfloat16* rh = cluster.map_shared_rank(w_hi, c) + c * per_cta;
      const __nv_bfloat16* rl = cluster.map_shared_rank(w_lo, c) + c * per_cta;
      for (int i = tid * 8; i < per_cta; i += LM_THREADS * 8) {
        *reinterpret_cast<uint4*>(w_hi + c * per_cta + i) = *reinterpret_cast<const uint4*>(rh + i);
        *reinterpret_cast<uint4*>(w_lo + c * per_cta + i) = *reinterpret_cast<const uint4*>(rl + i);
      }
    }
  }
  lm_cp_wait_all();                                            // this thread's part of the rows of A has landed
  cluster.sync();                                              // remote reads done (peers may exit); A visible to all warps

  // ---- phase 3: y += w A^T for this CTA's share of the outputs ---------------------------------------------------------------
  {
    const int kp = G >> 5;                                      // pairs of mma steps along G
    const __nv_bfloat16* As = reinterpret_cast<const __nv_bfloat16*>(stage);     // rows t_lo * 8 .. of A
    // the w fragments of the first 32 state rows do not depend on the output tile
    const uint4 wh_l = *reinterpret_cast<const uint4*>(w_hi + qrow * G + qcol * 8);
    const uint4 wh_h = *reinterpret_cast<const uint4*>(w_hi + (qrow + 8) * G + qcol * 8);
    const uint4 wl_l = *reinterpret_cast<const uint4*>(w_lo + qrow * G + qcol * 8);
    const uint4 wl_h = *reinterpret_cast<const uint4*>(w_lo + (qrow + 8) * G + qcol * 8);
    for (int t = t_lo + warp; t < t_hi; t += LM_WARPS) {
      const __nv_bfloat16* arow = As + (size_t)((t - t_lo) * 8 + qrow) * G + qcol * 8;
      const uint4 aw = *reinterpret_cast<const uint4*>(arow);
      uint32_t* py_lo = reinterpret_cast<uint32_t*>(ystage + (size_t)qrow * ys + (t - t_lo) * 16 + qcol * 4);
      uint32_t* py_hi = reinterpret_cast<uint32_t*>(ystage + (size_t)(qrow + 8) * ys + (t - t_lo) * 16 + qcol * 4);
      const uint32_t ylo = lo_ok ? *py_lo : 0u, yhi = hi_ok ? *py_hi : 0u;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
      lr_mma(c, wh_l.x, wh_h.x, wh_l.y, wh_h.y, aw.x, aw.y);
      lr_mma(c, wh_l.z, wh_h.z, wh_l.w, wh_h.w, aw.z, aw.w);
      lr_mma(c, wl_l.x, wl_h.x, wl_l.y, wl_h.y, aw.x, aw.y);
      lr_mma(c, wl_l.z, wl_h.z, wl_l.w, wl_h.w, aw.z, aw.w);
      for (int pp = 1; pp < kp; ++pp) {                         // more than 32 state rows
        const uint4 bw = *reinterpret_cast<const uint4*>(arow + pp * 32);
        const uint4 a_hl = *reinterpret_cast<const uint4*>(w_hi + qrow * G + pp * 32 + qcol * 8);
        const uint4 a_hh = *reinterpret_cast<const uint4*>(w_hi + (qrow + 8) * G + pp * 32 + qcol * 8);
        const uint4 a_ll = *reinterpret_cast<const uint4*>(w_lo + qrow * G + pp * 32 + qcol * 8);
        const uint4 a_lh = *reinterpret_cast<const uint4*>(w_lo + (qrow + 8) * G + pp * 32 + qcol * 8);
        lr_mma(c, a_hl.x, a_hh.x, a_hl.y, a_hh.y, bw.x, bw.y);
        lr_mma(c, a_hl.z, a_hh.z, a_hl.w, a_hh.w, bw.z, bw.w);
        lr_mma(c, a_ll.x, a_lh.x, a_ll.y, a_lh.y, bw.x, bw.y);
        lr_mma(c, a_ll.z, a_lh.z, a_ll.w, a_lh.w, bw.z, bw.w);
      }
      if (lo_ok) {
        const __nv_bfloat162 old = *reinterpret_cast<const __nv_bfloat162*>(&ylo);
        *py_lo = lr_pack(__low2float(old) + c[0], __high2float(old) + c[1]);
      }
      if (hi_ok) {
        const __nv_bfloat162 old = *reinterpret_cast<const __nv_bfloat162*>(&yhi);
        *py_hi = lr_pack(__low2float(old) + c[2], __high2float(old) + c[3]);
      }
    }
    __syncthreads();
    // the new outputs leave as whole 16-byte vectors, a warp per row
    const int yv = t_hi - t_lo;
    for (int row = warp; row < nseq; row += LM_WARPS) {
      if (active != nullptr && active[b0 + row] == 0) continue;
      for (int v = lane; v < yv; v += 32)
        *reinterpret_cast<uint4*>(yl + (size_t)row * d_out + (size_t)(t_lo + v) * 8) =
            *reinterpret_cast<const uint4*>(ystage + (size_t)row * ys + v * 16);
    }
  }
}

}  // namespace

cudaError_t ptenc_launch_lora_apply(ptenc_cache* c, int l0, int nl, const void* A, const void* Bm, const void* x,
                                    void* y, const uint8_t* active, int d_in, int d_out, cudaStream_t st) {
  const PtencDev& p = c->dev;
  // tensor-core path: bf16, r a multiple of 8, G and d_in multiples of 32 (d_in at least 128: a slice per CTA of the
  // cluster), d_out a multiple of 8, and slices that fit the staging buffer with two CTAs per SM
  if (c->cfg.dtype == PTENC_DTYPE_BF16 && (p.r & 7) == 0 && (p.G & 31) == 0 && (d_in & 31) == 0 && d_in >= 128 &&
      (d_out & 7) == 0 && lr_mma_smem(p.G, p.r, d_in, d_out) <= 100 * 1024 &&
      (long long)nl * ((p.B + LM_SEQ - 1) / LM_SEQ) <= 65535) {
    const size_t smem = lr_mma_smem(p.G, p.r, d_in, d_out);
    static bool attr_done_c[PTENC_MAX_DEVICES] = {};
    if (ptenc_first_use(attr_done_c, c->cfg.device)) {
      cudaError_t e = cudaFuncSetAttribute(k_lora_apply_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
      if (e != cudaSuccess) return e;
    }
    const int nb = (p.B + LM_SEQ - 1) / LM_SEQ;
    k_lora_apply_cluster<<<dim3(LM_CLUSTER, nl * nb), LM_THREADS, smem, st>>>(
        p, l0, (const __nv_bfloat16*)A, (const __nv_bfloat16*)Bm, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, active,
        d_in, d_out);
    c->launches++;
    return cudaGetLastError();
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
