// Per-record building blocks of the decode products: input staging with the fused token-shift
// mix (Appendix A.1 Eq. 20), and the record -> tensor-core step routines for both formats.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/rwkvq.h"
#include "unpack.cuh"

namespace rwkvq {

enum { FMT_SQ3 = 0, FMT_VQ6 = 1, FMT_VQ8 = 2 };

struct GemvArgs {
  const uint8_t* payload;   // chunks
  const uint8_t* aux;       // VQ codebooks
  const uint8_t* mu;        // vector index stream, or nullptr
  const uint8_t* mu_aux;    // vector codebook
  const __half* x;
  const __half* xprev;
  void* y;
  float* partial;
  unsigned* counters;
  int oc, ic, KT, S, nkt, entries, B, mu_bits, mu_entries, y_dtype;
};

struct SmemLayout {
  uint32_t xstride;   // bytes between batch rows of the staged input
  uint32_t gs_off;    // SQ: per-group sums  float[groups][3][16]
  uint32_t cb_off;    // VQ: two lane-replicated codebooks
  uint32_t mucb_off;  // token-shift codebook
  uint32_t total;
};

// Staged input rows are nkt*256 fp16 values plus 32 bytes of padding, which makes the 8-byte
// B-fragment loads of a half-warp (4 batch rows x 4 column quads) hit 16 distinct bank pairs.
__host__ __device__ inline SmemLayout smem_layout_rt(int fmt, int nkt, int B, int mu_entries, int entries) {
  SmemLayout L;
  L.xstride = (uint32_t)nkt * 512u + 32u;
  uint32_t off = (uint32_t)B * L.xstride;
  L.gs_off = off;
  if (fmt == FMT_SQ3) off += (uint32_t)nkt * 2u * 3u * 16u * 4u;
  off = (off + 127u) & ~127u;
  L.cb_off = off;
  if (fmt != FMT_SQ3) off += 2u * (uint32_t)entries * 128u;
  L.mucb_off = off;
  off += (uint32_t)mu_entries * 4u;
  L.total = (off + 15u) & ~15u;
  return L;
}
template <int FMT>
__host__ __device__ inline SmemLayout smem_layout(int nkt, int B, int mu_entries, int entries) {
  return smem_layout_rt(FMT, nkt, B, mu_entries, entries);
}

__device__ __forceinline__ uint32_t vector_index(const uint8_t* stream, int p, int bits) {
  const uint32_t bitpos = (uint32_t)p * (uint32_t)bits, byte = bitpos >> 3;
  const uint32_t v = (uint32_t)stream[byte] | ((uint32_t)stream[byte + 1] << 8);
  return (v >> (bitpos & 7u)) & ((1u << bits) - 1u);
}

__device__ __forceinline__ void store_y(void* y, int dtype, size_t idx, float v) {
  if (dtype == RWKVQ_F32) static_cast<float*>(y)[idx] = v;
  else static_cast<__half*>(y)[idx] = __float2half_rn(v);
}
__device__ __forceinline__ void store_w(void* out, int dtype, size_t idx, float v) {
  if (dtype == RWKVQ_F32) static_cast<float*>(out)[idx] = v;
  else static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(v);
}

// x_mix = x + (x_prev - x) * mu_hat for columns [kt0*256, kt1*256) of every batch row, rounded
// to fp16 into shared memory (zeros beyond ic); then, for SQ, per 128-column group and batch
// row the three sums the factored dequantisation needs:
//    Sx  = sum x,   Bx_h = sum bias_h(col) * x   (h = 0: rows g, 1: rows g+8 of a record)
// computed from the rounded values the tensor core will see, reduced with warp shuffles.
template <int FMT>
__device__ __forceinline__ void stage_input(uint8_t* smem, const SmemLayout& L, const GemvArgs& a, int kt0, int kt1) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  uint32_t* mucb = reinterpret_cast<uint32_t*>(smem + L.mucb_off);
  if (a.mu) {
    for (int e = tid; e < a.mu_entries; e += nthr) mucb[e] = reinterpret_cast<const uint32_t*>(a.mu_aux)[e];
    __syncthreads();
  }
  const int npairs = (kt1 - kt0) * 128;
  for (int p = tid; p < a.B * npairs; p += nthr) {
    const int b = p / npairs, cp = p - b * npairs;
    const int col = kt0 * 256 + 2 * cp;
    __half2 v = __float2half2_rn(0.f);
    if (col < a.ic) {
      v = *reinterpret_cast<const __half2*>(a.x + (size_t)b * a.ic + col);
      if (a.mu) {
        const float2 xf = __half22float2(v);
        const float2 pf = __half22float2(*reinterpret_cast<const __half2*>(a.xprev + (size_t)b * a.ic + col));
        const uint32_t mw = mucb[vector_index(a.mu, col >> 1, a.mu_bits)];
        const float2 mf = __half22float2(*reinterpret_cast<const __half2*>(&mw));
        v = __floats2half2_rn(fmaf(pf.x - xf.x, mf.x, xf.x), fmaf(pf.y - xf.y, mf.y, xf.y));
      }
    }
    *reinterpret_cast<__half2*>(smem + (size_t)b * L.xstride + (size_t)cp * 4) = v;
  }
  __syncthreads();
  if constexpr (FMT == FMT_SQ3) {
    const int lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
    const int ngroups = (kt1 - kt0) * 2;
    float* gs = reinterpret_cast<float*>(smem + L.gs_off);
    const int o = (lane * 4) & 63;
    const float b00 = (float)rwkvq_sq_bias(o, 0), b02 = (float)rwkvq_sq_bias(o + 2, 0);
    const float b10 = (float)rwkvq_sq_bias(o, 1), b12 = (float)rwkvq_sq_bias(o + 2, 1);
    for (int task = warp; task < ngroups * a.B; task += nwarps) {
      const int grp = task / a.B, b = task - grp * a.B;
      const uint2 raw = *reinterpret_cast<const uint2*>(smem + (size_t)b * L.xstride + (size_t)(grp * 128 + lane * 4) * 2);
      const float2 x01 = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
      const float2 x23 = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
      const float p01 = x01.x + x01.y, p23 = x23.x + x23.y;
      float sx = p01 + p23;
      float s0 = fmaf(b00, p01, b02 * p23);
      float s1 = fmaf(b10, p01, b12 * p23);
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) {
        sx += __shfl_xor_sync(0xFFFFFFFFu, sx, d);
        s0 += __shfl_xor_sync(0xFFFFFFFFu, s0, d);
        s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, d);
      }
      if (lane == 0) {
        gs[(grp * 3 + 0) * 16 + b] = sx;
        gs[(grp * 3 + 1) * 16 + b] = s0;
        gs[(grp * 3 + 2) * 16 + b] = s1;
      }
    }
    __syncthreads();
  }
}

// Per-lane view of the staged input for one 256-column tile.  Lane (g, t) of a warp reads, for
// tensor-core step j and batch block n, the 8 bytes x_mix[8n + g][16j + 4t .. +3]; `x[n]` points at
// step 0 of that row, so a fragment is one 64-bit load at a compile-time offset.  Batch rows beyond
// B are clamped to row B-1: the tensor core then computes values for batch columns that do not
// exist, which are never stored.  `gs` points at the sums (Sx, Bx_0, Bx_1) of the tile's first group
// for batch columns 2t, 2t+1; the three rows are `gstride` bytes apart and groups 3*gstride.
struct XLane {
  const uint8_t* x[2];
  const uint8_t* gs;
  uint32_t gstride;
};

// xtile: first column of the tile in batch row 0; rows `xstride` bytes apart.  gs_tile: sums of the
// tile's first group, laid out [group][3][nbp] floats.
__device__ __forceinline__ XLane make_xlane(const uint8_t* xtile, uint32_t xstride, const float* gs_tile, uint32_t nbp,
                                            int B, int lane) {
  const int g = lane >> 2, t = lane & 3;
  XLane xl;
  xl.x[0] = xtile + (size_t)min(g, B - 1) * xstride + t * 8;
  xl.x[1] = xtile + (size_t)min(8 + g, B - 1) * xstride + t * 8;
  xl.gs = reinterpret_cast<const uint8_t*>(gs_tile) + t * 8;
  xl.gstride = nbp * 4u;
  return xl;
}

struct SqRecord {
  uint4 p0, p1, p2, sz;
  __device__ __forceinline__ void load_shared(const uint8_t* rec, int lane) {
    p0 = *reinterpret_cast<const uint4*>(rec + lane * 16);
    p1 = *reinterpret_cast<const uint4*>(rec + 512 + lane * 16);
    p2 = *reinterpret_cast<const uint4*>(rec + 1024 + lane * 16);
    sz = *reinterpret_cast<const uint4*>(rec + RWKVQ_SQ_CODE_BYTES + (lane >> 2) * 16);
  }
  __device__ __forceinline__ void load(const uint8_t* rec, int lane) {
    p0 = ldg_stream(rec + lane * 16);
    p1 = ldg_stream(rec + 512 + lane * 16);
    p2 = ldg_stream(rec + 1024 + lane * 16);
    sz = ldg_stream(rec + RWKVQ_SQ_CODE_BYTES + (lane >> 2) * 16);
  }
  __device__ __forceinline__ void words(uint32_t (&w)[12]) const {
    w[0] = p0.x; w[1] = p0.y; w[2] = p0.z; w[3] = p0.w;
    w[4] = p1.x; w[5] = p1.y; w[6] = p1.z; w[7] = p1.w;
    w[8] = p2.x; w[9] = p2.y; w[10] = p2.z; w[11] = p2.w;
  }
  // k = 2 * row_half + group:  low 16 bits = s, high 16 bits = z (fp16)
  __device__ __forceinline__ uint32_t sz_word(int k) const { return k == 0 ? sz.x : k == 1 ? sz.y : k == 2 ? sz.z : sz.w; }
};

// One 128-column group of an SQ record (16 rows) against the staged input:
//   y[b][row] += s * ( sum_cols (q+bias) x  -  Bx_h  -  z * Sx )
// The inner sum is eight m16n8k16 steps with fp32 accumulation in the tensor core; the bias each
// extracted half carries is removed with the precomputed Bx_h.  `w` holds the group's six words
// (two triples), `sz_lo` / `sz_hi` the (s, z) fp16 pairs of rows g and g+8.  GRP selects the
// 128-column half of the tile `xl` describes.
template <int NB, int GRP>
__device__ __forceinline__ void sq_group_mma(const uint32_t (&w)[6], uint32_t sz_lo, uint32_t sz_hi, const XLane& xl,
                                             float (&acc)[NB][4]) {
  float c[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n) c[n][0] = c[n][1] = c[n][2] = c[n][3] = 0.f;
#pragma unroll
  for (int ti = 0; ti < 2; ++ti) {
    uint32_t r[16];
    sq_unpack_triple(w[3 * ti], w[3 * ti + 1], w[3 * ti + 2], r);
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const uint32_t afrag[4] = {r[4 * m], r[4 * m + 1], r[4 * m + 2], r[4 * m + 3]};
#pragma unroll
      for (int n = 0; n < NB; ++n) {
        const uint2 bf = *reinterpret_cast<const uint2*>(xl.x[n] + GRP * 256 + (4 * ti + m) * 32);
        mma_16816(c[n], afrag, bf.x, bf.y);
      }
    }
  }
  const float2 sz0 = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));
  const float2 sz1 = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));
  const uint8_t* gsp = xl.gs + (size_t)(GRP * 3) * xl.gstride;
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const float2 sx = *reinterpret_cast<const float2*>(gsp + n * 32);
    const float2 b0 = *reinterpret_cast<const float2*>(gsp + xl.gstride + n * 32);
    const float2 b1 = *reinterpret_cast<const float2*>(gsp + 2 * xl.gstride + n * 32);
    acc[n][0] = fmaf(sz0.x, fmaf(-sz0.y, sx.x, c[n][0] - b0.x), acc[n][0]);
    acc[n][1] = fmaf(sz0.x, fmaf(-sz0.y, sx.y, c[n][1] - b0.y), acc[n][1]);
    acc[n][2] = fmaf(sz1.x, fmaf(-sz1.y, sx.x, c[n][2] - b1.x), acc[n][2]);
    acc[n][3] = fmaf(sz1.x, fmaf(-sz1.y, sx.y, c[n][3] - b1.y), acc[n][3]);
  }
}

// A whole SQ record (16 rows x 256 columns): its two groups in turn.
template <int NB>
__device__ __forceinline__ void sq_record_mma(const uint32_t (&w)[12], const uint4 sz, const XLane& xl,
                                              float (&acc)[NB][4]) {
  const uint32_t w0[6] = {w[0], w[1], w[2], w[3], w[4], w[5]};
  const uint32_t w1[6] = {w[6], w[7], w[8], w[9], w[10], w[11]};
  sq_group_mma<NB, 0>(w0, sz.x, sz.z, xl, acc);
  sq_group_mma<NB, 1>(w1, sz.y, sz.w, xl, acc);
}

// Two SQ records that cover the same 128 columns (rows r and r + 128 of a 256-row tile): every
// input fragment is loaded once and used by both.  `wa` / `wb`: the group's six words of each
// record; sza / szb: the records' (s, z) words {row g group 0, row g group 1, row g+8 group 0,
// row g+8 group 1}.  has_b == false skips the second record (warp-uniform).
template <int NB, int GRP>
__device__ __forceinline__ void sq_group_mma2(const uint32_t (&wa)[6], const uint32_t (&wb)[6], const uint4 sza,
                                              const uint4 szb, bool has_b, const XLane& xl, float (&acca)[NB][4],
                                              float (&accb)[NB][4]) {
  // The tensor-core chains start at -Bx_h, the bias the extracted halves carry, instead of at zero:
  // what they end with is sum(q x) of the group.
  const uint8_t* gsp = xl.gs + (size_t)(GRP * 3) * xl.gstride;
  float ca[NB][4], cb[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const float2 b0 = *reinterpret_cast<const float2*>(gsp + xl.gstride + n * 32);
    const float2 b1 = *reinterpret_cast<const float2*>(gsp + 2 * xl.gstride + n * 32);
    ca[n][0] = cb[n][0] = -b0.x; ca[n][1] = cb[n][1] = -b0.y;
    ca[n][2] = cb[n][2] = -b1.x; ca[n][3] = cb[n][3] = -b1.y;
  }
#pragma unroll
  for (int ti = 0; ti < 2; ++ti) {
    uint2 bf[4][NB];
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
      for (int n = 0; n < NB; ++n) bf[m][n] = *reinterpret_cast<const uint2*>(xl.x[n] + GRP * 256 + (4 * ti + m) * 32);
    {
      uint32_t r[16];
      sq_unpack_triple(wa[3 * ti], wa[3 * ti + 1], wa[3 * ti + 2], r);
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        const uint32_t afrag[4] = {r[4 * m], r[4 * m + 1], r[4 * m + 2], r[4 * m + 3]};
#pragma unroll
        for (int n = 0; n < NB; ++n) mma_16816(ca[n], afrag, bf[m][n].x, bf[m][n].y);
      }
    }
    if (has_b) {
      uint32_t r[16];
      sq_unpack_triple(wb[3 * ti], wb[3 * ti + 1], wb[3 * ti + 2], r);
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        const uint32_t afrag[4] = {r[4 * m], r[4 * m + 1], r[4 * m + 2], r[4 * m + 3]};
#pragma unroll
        for (int n = 0; n < NB; ++n) mma_16816(cb[n], afrag, bf[m][n].x, bf[m][n].y);
      }
    }
  }
  const uint32_t a_lo = GRP == 0 ? sza.x : sza.y, a_hi = GRP == 0 ? sza.z : sza.w;
  const uint32_t b_lo = GRP == 0 ? szb.x : szb.y, b_hi = GRP == 0 ? szb.z : szb.w;
  const float2 sa0 = __half22float2(*reinterpret_cast<const __half2*>(&a_lo));
  const float2 sa1 = __half22float2(*reinterpret_cast<const __half2*>(&a_hi));
  const float2 sb0 = __half22float2(*reinterpret_cast<const __half2*>(&b_lo));
  const float2 sb1 = __half22float2(*reinterpret_cast<const __half2*>(&b_hi));
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const float2 sx = *reinterpret_cast<const float2*>(gsp + n * 32);
    acca[n][0] = fmaf(sa0.x, fmaf(-sa0.y, sx.x, ca[n][0]), acca[n][0]);
    acca[n][1] = fmaf(sa0.x, fmaf(-sa0.y, sx.y, ca[n][1]), acca[n][1]);
    acca[n][2] = fmaf(sa1.x, fmaf(-sa1.y, sx.x, ca[n][2]), acca[n][2]);
    acca[n][3] = fmaf(sa1.x, fmaf(-sa1.y, sx.y, ca[n][3]), acca[n][3]);
    accb[n][0] = fmaf(sb0.x, fmaf(-sb0.y, sx.x, cb[n][0]), accb[n][0]);
    accb[n][1] = fmaf(sb0.x, fmaf(-sb0.y, sx.y, cb[n][1]), accb[n][1]);
    accb[n][2] = fmaf(sb1.x, fmaf(-sb1.y, sx.x, cb[n][2]), accb[n][2]);
    accb[n][3] = fmaf(sb1.x, fmaf(-sb1.y, sx.y, cb[n][3]), accb[n][3]);
  }
}

template <int BITS>
struct VqRecord {
  static constexpr int NW = 2 * BITS;  // 64 indices of BITS bits = 2*BITS words per lane
  uint32_t w[NW];
  __device__ __forceinline__ void load_shared(const uint8_t* rec, int lane) {
#pragma unroll
    for (int p = 0; p < NW / 4; ++p) {
      const uint4 v = *reinterpret_cast<const uint4*>(rec + p * 512 + lane * 16);
      w[4 * p] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
    }
  }
  __device__ __forceinline__ void load(const uint8_t* rec, int lane) {
#pragma unroll
    for (int p = 0; p < NW / 4; ++p) {
      const uint4 v = ldg_stream(rec + p * 512 + lane * 16);
      w[4 * p] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
    }
  }
};

// Copy one codebook (E half2 entries) into 32 lane-private replicas: entry e of lane l at word
// e*32 + l, so a lookup by any index pattern is bank-conflict free.
__device__ __forceinline__ void stage_codebook(uint8_t* dst, const uint32_t* src, int E) {
  uint32_t* d = reinterpret_cast<uint32_t*>(dst);
  for (int idx = threadIdx.x; idx < E * 32; idx += blockDim.x) d[idx] = __ldg(src + (idx >> 5));
}

// One VQ record: every fragment register is one codebook lookup (a 2-D vector is exactly the
// (even, odd) column pair a fragment register holds).
template <int BITS, int NB, int JBEG = 0, int JEND = 16>
__device__ __forceinline__ void vq_record_mma(const uint32_t (&w)[2 * BITS], const uint32_t* cb_lane, const XLane& xl,
                                              float (&acc)[NB][4]) {
#pragma unroll
  for (int j = JBEG; j < JEND; ++j) {
    uint32_t afrag[4];
#pragma unroll
    for (int R = 0; R < 4; ++R) afrag[R] = cb_lane[vq_index<BITS, 2 * BITS>(w, 4 * j + R) * 32u];
#pragma unroll
    for (int n = 0; n < NB; ++n) {
      const uint2 bf = *reinterpret_cast<const uint2*>(xl.x[n] + j * 32);
      mma_16816(acc[n], afrag, bf.x, bf.y);
    }
  }
}

// Words [HALF * BITS, (HALF + 1) * BITS) of a lane's VQ stream (the indices of eight tensor-core
// steps) from a record in shared memory; the other entries of `w` are left untouched.
template <int BITS, int HALF>
__device__ __forceinline__ void vq_half_words(const uint8_t* rec, int lane, uint32_t (&w)[2 * BITS]) {
  if constexpr (BITS == 8) {
    const uint4 p = *reinterpret_cast<const uint4*>(rec + (2 * HALF) * 512 + lane * 16);
    const uint4 q = *reinterpret_cast<const uint4*>(rec + (2 * HALF + 1) * 512 + lane * 16);
    w[8 * HALF + 0] = p.x; w[8 * HALF + 1] = p.y; w[8 * HALF + 2] = p.z; w[8 * HALF + 3] = p.w;
    w[8 * HALF + 4] = q.x; w[8 * HALF + 5] = q.y; w[8 * HALF + 6] = q.z; w[8 * HALF + 7] = q.w;
  } else if constexpr (HALF == 0) {
    const uint4 p = *reinterpret_cast<const uint4*>(rec + lane * 16);
    const uint2 q = *reinterpret_cast<const uint2*>(rec + 512 + lane * 16);
    w[0] = p.x; w[1] = p.y; w[2] = p.z; w[3] = p.w; w[4] = q.x; w[5] = q.y;
  } else {
    const uint2 p = *reinterpret_cast<const uint2*>(rec + 512 + lane * 16 + 8);
    const uint4 q = *reinterpret_cast<const uint4*>(rec + 1024 + lane * 16);
    w[6] = p.x; w[7] = p.y; w[8] = q.x; w[9] = q.y; w[10] = q.z; w[11] = q.w;
  }
}

// Eight tensor-core steps (HALF of the tile's columns) of two VQ records of one tile (rows r and
// r + 128, same columns, same codebook): shared input fragments, eight lookups per step.
template <int BITS, int NB, int HALF>
__device__ __forceinline__ void vq_half_mma2(const uint32_t (&wa)[2 * BITS], const uint32_t (&wb)[2 * BITS],
                                             const uint32_t* cb_lane, const XLane& xl, float (&acca)[NB][4],
                                             float (&accb)[NB][4]) {
#pragma unroll
  for (int j = 8 * HALF; j < 8 * HALF + 8; ++j) {
    uint32_t fa[4], fb[4];
#pragma unroll
    for (int R = 0; R < 4; ++R) {
      fa[R] = cb_lane[vq_index<BITS, 2 * BITS>(wa, 4 * j + R) * 32u];
      fb[R] = cb_lane[vq_index<BITS, 2 * BITS>(wb, 4 * j + R) * 32u];
    }
#pragma unroll
    for (int n = 0; n < NB; ++n) {
      const uint2 bf = *reinterpret_cast<const uint2*>(xl.x[n] + j * 32);
      mma_16816(acca[n], fa, bf.x, bf.y);
      mma_16816(accb[n], fb, bf.x, bf.y);
    }
  }
}

inline void fill_gemv_args(GemvArgs* a, const rwkvq_desc* d, const void* W, const rwkvq_desc* mud, const void* mu,
                           const void* x, const void* xprev, int B, void* y, int y_dtype) {
  const uint8_t* img = static_cast<const uint8_t*>(W);
  size_t rb = d->method == RWKVQ_SQ ? RWKVQ_SQ_RECORD_BYTES : rwkvq_vq_record_bytes(d->bits);
  a->payload = img + RWKVQ_HEADER_BYTES;
  a->aux = img + RWKVQ_HEADER_BYTES + (size_t)(d->oc_pad / 128) * (d->ic_pad / 256) * 8 * rb;
  a->mu = nullptr; a->mu_aux = nullptr; a->mu_bits = 0; a->mu_entries = 0;
  if (mu) {
    const uint8_t* m = static_cast<const uint8_t*>(mu);
    a->mu = m + RWKVQ_HEADER_BYTES;
    a->mu_aux = m + RWKVQ_HEADER_BYTES + ((((size_t)(mud->ic / 2) * mud->bits + 7) / 8 + 15) / 16 * 16);
    a->mu_bits = mud->bits; a->mu_entries = mud->entries;
  }
  a->x = static_cast<const __half*>(x);
  a->xprev = static_cast<const __half*>(xprev);
  a->y = y; a->partial = nullptr; a->counters = nullptr;
  a->oc = d->oc; a->ic = d->ic; a->entries = d->entries; a->B = B; a->y_dtype = y_dtype;
  a->KT = d->ic_pad / 256; a->S = 1; a->nkt = a->KT;
}

}  // namespace rwkvq
