// Device quantizers: the round-to-nearest scalar quantizer of Section 3.2 Eq. 2, the k-means
// vector quantizer of Section 3.2 Eq. 3 (one codebook per 256 x 256 tile, or per token-shift
// vector), the X^2-weighted k-means of Section 4.2 Eq. 19 for token-shift vectors, and the
// percentile-clipped representative activation of Section 4.2.  Each writes the packed device
// image of format.h directly; nothing passes through the host.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rwkvq.h"
#include "format.h"
#include "host_util.h"

namespace rwkvq {
namespace {

constexpr int kFlagNonFinite = 1;

// ---- scalar quantizer ------------------------------------------------------------------------
//
// One warp per record (16 rows x 256 columns), one block of eight warps per chunk.  Pass 1 finds
// each (row, group) minimum and maximum with packed fp16 min/max and shuffles (lanes 0..15 hold
// group 0, lanes 16..31 group 1, eight columns each); lane r + 16 h then derives (s, z) of
// (row r, group h) in fp64 exactly as Eq. 2 prescribes.
//
// The codes need no division.  q = clamp(round(w / s) + z, 0, 7) counts the k in 1..7 with
// round(w / s) >= k - z, and round(x) >= m (ties to even) holds iff x > m - 1/2, or x = m - 1/2
// with m even.  (m - 1/2) * s is exact in fp32 (4 bits times 11 bits), so each k has an exact
// fp16 threshold T_k -- the smallest fp16 number that is >= (or >) that product -- and
// q = #{k : w >= T_k}, seven packed fp16 comparisons for two weights.  Pass 2 reads the rows
// again (from cache) and counts.
constexpr int kSqRowStride = 256 + 16;   // bytes per row of the code staging area: conflict-free lane reads

__device__ __forceinline__ float h2f_bits(uint32_t h) { return __half2float(__ushort_as_half((unsigned short)h)); }
__device__ __forceinline__ __half2 as_h2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }
__device__ __forceinline__ uint32_t as_u32(__half2 v) { return *reinterpret_cast<uint32_t*>(&v); }

__global__ void __launch_bounds__(256, 3) sq_quantize_kernel(const uint16_t* __restrict__ w, int oc, int ic, int KT,
                                                             uint8_t* __restrict__ payload, int* __restrict__ flags) {
  __shared__ __align__(16) uint8_t codes_all[8][16 * kSqRowStride];
  __shared__ __align__(16) uint32_t thr_all[8][2][16][8];     // [warp][group][row][k]: (T_k, T_k) as half2, k = 1..7 in 0..6
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mb = blockIdx.x / KT, kt = blockIdx.x % KT;
  const int r0 = mb * 128 + warp * 16, c0 = kt * 256;
  uint8_t* codes = codes_all[warp];
  const int half = lane >> 4;
  const int col = c0 + 8 * lane;
  const bool col_in = col < ic;            // ic is a multiple of 128: a whole group is inside or outside
  const uint16_t* src = w + (size_t)r0 * ic + col;
  float my_mn = 0.f, my_mx = 0.f;
  uint32_t bad = 0u;
#pragma unroll 4
  for (int r = 0; r < 16; ++r) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (col_in && r0 + r < oc) v = __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * ic));
    // an all-ones exponent carries into bit 15 of its half
    bad |= ((v.x & 0x7C007C00u) + 0x04000400u) | ((v.y & 0x7C007C00u) + 0x04000400u) |
           ((v.z & 0x7C007C00u) + 0x04000400u) | ((v.w & 0x7C007C00u) + 0x04000400u);
    __half2 mn2 = __hmin2(__hmin2(as_h2(v.x), as_h2(v.y)), __hmin2(as_h2(v.z), as_h2(v.w)));
    __half2 mx2 = __hmax2(__hmax2(as_h2(v.x), as_h2(v.y)), __hmax2(as_h2(v.z), as_h2(v.w)));
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) {
      mn2 = __hmin2(mn2, as_h2(__shfl_xor_sync(0xFFFFFFFFu, as_u32(mn2), off)));
      mx2 = __hmax2(mx2, as_h2(__shfl_xor_sync(0xFFFFFFFFu, as_u32(mx2), off)));
    }
    if ((lane & 15) == r) {
      my_mn = fminf(__low2float(mn2), __high2float(mn2));
      my_mx = fmaxf(__low2float(mx2), __high2float(mx2));
    }
  }
  if (bad & 0x80008000u) atomicOr(flags, kFlagNonFinite);
  // (s, z) of (row lane & 15, group half), Eq. 2; a constant group c is coded exactly:
  // c == 0 -> (1, 0, q 0), c > 0 -> (c, 0, q 1), c < 0 -> (|c|, 1, q 0).
  float my_s, my_z;
  {
    const double mn = (double)my_mn, mx = (double)my_mx;
    const __half s16 = __double2half((mx - mn) / 7.0);
    const double s = (double)__half2float(s16);
    uint32_t* thr = thr_all[warp][half][lane & 15];
    const uint32_t kNever = 0x7C007C00u, kAlways = 0xFC00FC00u;     // +inf, -inf
    if (mx == mn || s == 0.0) {
      my_s = mn == 0.0 ? 1.f : fabsf(my_mn);
      my_z = mn < 0.0 ? 1.f : 0.f;
      thr[0] = mn > 0.0 ? kAlways : kNever;
#pragma unroll
      for (int k = 1; k < 7; ++k) thr[k] = kNever;
    } else {
      my_s = (float)s;
      my_z = (float)fmin(7.0, fmax(0.0, rint(-mn / s)));
#pragma unroll
      for (int k = 1; k <= 7; ++k) {
        const float m = (float)k - my_z;
        const float theta = (m - 0.5f) * my_s;                  // exact
        __half t16 = __float2half_ru(theta);                   // smallest fp16 >= theta (+inf / -65504 beyond the range)
        if (((int)m & 1) && __half2float(t16) == theta) {       // m odd: the tie rounds down, so w must exceed theta
          const unsigned short hb = __half_as_ushort(t16);
          t16 = __ushort_as_half((hb & 0x7FFFu) == 0 ? (unsigned short)1 : (hb & 0x8000u) ? (unsigned short)(hb - 1) : (unsigned short)(hb + 1));
        }
        const uint32_t tb = __half_as_ushort(t16);
        thr[k - 1] = tb | (tb << 16);
      }
    }
    thr[7] = 0u;
  }
  __syncwarp();
#pragma unroll 4
  for (int r = 0; r < 16; ++r) {
    const bool inside = col_in && (r0 + r) < oc;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (inside) v = __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * ic));
    const uint4 ta = *reinterpret_cast<const uint4*>(thr_all[warp][half][r]);
    const uint4 tb = *reinterpret_cast<const uint4*>(thr_all[warp][half][r] + 4);
    const uint32_t words[4] = {v.x, v.y, v.z, v.w};
    uint32_t qw[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const __half2 x = as_h2(words[k]);
      __half2 acc = as_h2(0x64006400u);       // 1024: the count appears in the low mantissa bits
      acc = __hadd2(acc, __hge2(x, as_h2(ta.x)));
      acc = __hadd2(acc, __hge2(x, as_h2(ta.y)));
      acc = __hadd2(acc, __hge2(x, as_h2(ta.z)));
      acc = __hadd2(acc, __hge2(x, as_h2(ta.w)));
      acc = __hadd2(acc, __hge2(x, as_h2(tb.x)));
      acc = __hadd2(acc, __hge2(x, as_h2(tb.y)));
      acc = __hadd2(acc, __hge2(x, as_h2(tb.z)));
      qw[k] = as_u32(acc) & 0x00070007u;
    }
    const uint2 out = make_uint2(__byte_perm(qw[0], qw[1], 0x6420u), __byte_perm(qw[2], qw[3], 0x6420u));
    *reinterpret_cast<uint2*>(codes + r * kSqRowStride + 8 * lane) = inside ? out : make_uint2(0u, 0u);
  }
  __syncwarp();
  // Bit packing of format.h: lane (g, t) owns rows g and g + 8 and, in every tensor-core step,
  // the four columns 4t .. 4t+3 (one 32-bit read of the staging area = registers R and R + 2).
  const int g = lane >> 2, t = lane & 3;
  uint8_t* rec = payload + ((size_t)blockIdx.x * 8 + warp) * RWKVQ_SQ_RECORD_BYTES;
  uint32_t wd[12];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t w3[3] = {0u, 0u, 0u};
#pragma unroll
    for (int m = 0; m < 4; ++m) {
#pragma unroll
      for (int hrow = 0; hrow < 2; ++hrow) {
        const uint32_t four = *reinterpret_cast<const uint32_t*>(codes + (g + 8 * hrow) * kSqRowStride + 64 * i + 16 * m + 4 * t);
#pragma unroll
        for (int cp = 0; cp < 2; ++cp) {
          const int e = 4 * m + 2 * cp + hrow;             // register R = 2 * cp + hrow of step m
          const uint32_t pair = __byte_perm(four, 0u, cp ? 0x4342u : 0x4140u);   // (even column) | (odd column) << 16
          if (e < 15) {
            w3[e / 5] |= pair << (3 * (e % 5));
          } else {
#pragma unroll
            for (int b = 0; b < 3; ++b) w3[b] |= ((pair >> b) & 0x00010001u) << 15;
          }
        }
      }
    }
    wd[3 * i] = w3[0]; wd[3 * i + 1] = w3[1]; wd[3 * i + 2] = w3[2];
  }
#pragma unroll
  for (int p = 0; p < 3; ++p)
    *reinterpret_cast<uint4*>(rec + p * 512 + lane * 16) = make_uint4(wd[4 * p], wd[4 * p + 1], wd[4 * p + 2], wd[4 * p + 3]);
  // plane 3: for g = 0..7 the (s, z) pairs of (row g, group 0), (row g, group 1), (row g+8, group 0), (row g+8, group 1)
  {
    const int r = lane & 15;
    const bool inside = (r0 + r) < oc && (c0 + 128 * half) < ic;
    const uint32_t s_bits = inside ? (uint32_t)__half_as_ushort(__float2half_rn(my_s)) : 0u;
    const uint32_t z_bits = inside ? (uint32_t)__half_as_ushort(__float2half_rn(my_z)) : 0u;
    *reinterpret_cast<uint32_t*>(rec + RWKVQ_SQ_CODE_BYTES + (r & 7) * 16 + ((r >> 3) * 2 + half) * 4) = s_bits | (z_bits << 16);
  }
}

// ---- vector quantizer ------------------------------------------------------------------------
//
// One block of 512 threads per codebook: a 256 x 256 tile (32768 two-element vectors, vector
// i = 128 * row + pair) or one token-shift vector (ic / 2 vectors).  The vectors stay in shared
// memory as fp16 pairs; thread t owns vectors 64 t .. 64 t + 63, so that a scan over threads is a
// scan over vector numbers.
constexpr int kVqThreads = 512;
constexpr int kVqPerThread = 64;
constexpr int kVqMaxVec = kVqThreads * kVqPerThread;   // 32768
constexpr int kVqMaxE = 256;

struct SplitMix64 {   // Steele, Lea, Flood: "Fast splittable pseudorandom number generators" (2014)
  uint64_t s;
  __device__ uint64_t next() {
    uint64_t z = (s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  }
};

struct VqShared {
  double cx[kVqMaxE], cy[kVqMaxE];            // centres
  unsigned long long sx[kVqMaxE], sy[kVqMaxE];  // exact sums of members, in units of 2^-24 (two's complement)
  unsigned int cnt[kVqMaxE];
  float2 cf[kVqMaxE];                         // centres rounded to fp32 for the assignment
  float warp_tot[kVqThreads / 32];
  uint64_t draw[2];                           // double-buffered by the parity of the seeding round
  int pick[2];
};

struct VqArgs {
  const uint16_t* w;        // matrix [oc][ic] or vector [ic]
  const float* elem_w;      // vector mode: X^2 per element, or NULL
  int ic;                   // row length of w
  int TC;                   // tiles per row of tiles (matrix mode)
  int n_vec;                // vectors per codebook
  int bits, E, iters;
  int is_vector;
  uint64_t seed;
  uint8_t* payload;         // matrix: chunk grid; vector: bit stream
  uint32_t* aux;            // codebooks, E half2 each
  int* flags;
};

// fp16 value times 2^24 as an exact integer (|v| < 2^16, multiples of 2^-24)
__device__ __forceinline__ long long half_fixed(uint32_t h) {
  const int e = (h >> 10) & 31, m = h & 1023;
  const long long mag = e ? ((long long)(m + 1024) << (e - 1)) : (long long)m;
  return (h & 0x8000u) ? -mag : mag;
}

// Inclusive scan of the per-thread sums of `dist` in thread order; returns the total.  The
// thread whose range [excl, incl) holds u01 * total walks its vectors for the first running sum
// above the target and publishes that vector's number in *pick_out.
__device__ __forceinline__ float block_scan_pick(VqShared& sh, const float (&dist)[kVqPerThread], int n_mine, int base,
                                                 float u01, int* pick_out) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float local = 0.f;
#pragma unroll
  for (int k = 0; k < kVqPerThread; ++k) local += (k < n_mine) ? dist[k] : 0.f;
  float incl = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const float v = __shfl_up_sync(0xFFFFFFFFu, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) sh.warp_tot[warp] = incl;
  __syncthreads();
  float before = 0.f, total = 0.f;
  for (int wv = 0; wv < kVqThreads / 32; ++wv) {
    if (wv == warp) before = total;
    total += sh.warp_tot[wv];
  }
  float excl_in_warp = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
  if (lane == 0) excl_in_warp = 0.f;
  const float excl = before + excl_in_warp, inc = before + incl;
  const float target = u01 * total;
  if (total > 0.f && excl <= target && target < inc) {
    float acc = excl;
    int pick = base;
#pragma unroll
    for (int k = 0; k < kVqPerThread; ++k) {
      if (k < n_mine) {
        const bool begins_below = acc <= target;
        acc += dist[k];
        if (begins_below) pick = base + k;      // last vector whose running sum began at or below the target
      }
    }
    *pick_out = pick;
  }
  __syncthreads();
  return total;
}

// storage position of vector i: thread t = i / 64 owns a row of 64 words; the row is rotated by
// the lane so that the lanes of a warp, which walk their rows in step, hit different banks
__device__ __forceinline__ int vq_slot(int i) { return (i & ~63) | ((i ^ (i >> 6)) & 31) | (i & 32); }

__device__ __forceinline__ float d2f(float x, float y, float2 c) {
  const float dx = x - c.x, dy = y - c.y;
  return fmaf(dx, dx, dy * dy);
}

// The 64 indices of lane (g, t) of record `rec` of the tile as its little-endian bit stream.
template <int BITS>
__device__ __forceinline__ void vq_pack_lane(const uint8_t* idx, int rec, int g, int t, int L, uint8_t* out) {
  uint32_t words[2 * BITS + 1];
#pragma unroll
  for (int k = 0; k < 2 * BITS + 1; ++k) words[k] = 0u;
#pragma unroll
  for (int nn = 0; nn < 64; ++nn) {
    const int j = nn >> 2, R = nn & 3;
    const int row = rec * 16 + g + 8 * (R & 1);
    const int pair = 8 * j + 2 * t + (R >> 1);
    const uint32_t v = idx[row * 128 + pair];
    const int bitpos = BITS * nn, wi = bitpos >> 5, shft = bitpos & 31;
    words[wi] |= v << shft;
    if (shft + BITS > 32) words[wi + 1] |= v >> (32 - shft);
  }
#pragma unroll
  for (int p = 0; p < BITS / 2; ++p)
    *reinterpret_cast<uint4*>(out + p * 512 + L * 16) = make_uint4(words[4 * p], words[4 * p + 1], words[4 * p + 2], words[4 * p + 3]);
}

__global__ void __launch_bounds__(kVqThreads, 1) vq_kmeans_kernel(const VqArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint32_t* vec = reinterpret_cast<uint32_t*>(smem);
  uint8_t* idx = smem + (size_t)kVqMaxVec * 4;
  VqShared& sh = *reinterpret_cast<VqShared*>(smem + (size_t)kVqMaxVec * 5);
  const int tid = threadIdx.x;
  const int tile = blockIdx.x;
  const int tr = a.is_vector ? 0 : tile / a.TC, tc = a.is_vector ? 0 : tile % a.TC;
  const int n = a.n_vec, E = a.E;
  const bool weighted = a.elem_w != nullptr;
  {
    bool bad = false;
    for (int i = tid; i < kVqMaxVec; i += kVqThreads) {
      uint32_t v = 0u;
      if (i < n) {
        const uint32_t* src = a.is_vector ? reinterpret_cast<const uint32_t*>(a.w) + i
            : reinterpret_cast<const uint32_t*>(a.w + (size_t)(tr * 256 + (i >> 7)) * a.ic + tc * 256) + (i & 127);
        v = __ldg(src);
        bad |= ((v & 0x7C00u) == 0x7C00u) | ((v & 0x7C000000u) == 0x7C000000u);
      }
      vec[vq_slot(i)] = v;
    }
    if (bad) atomicOr(a.flags, kFlagNonFinite);
  }
  const int base = tid * kVqPerThread;
  const int n_mine = max(0, min(kVqPerThread, n - base));
  SplitMix64 rng;
  rng.s = a.is_vector ? a.seed : a.seed * 0x9E3779B97F4A7C15ull + (uint64_t)tile + 1ull;
  auto below = [&](uint64_t r) {
    return (int)((unsigned long long)((double)(r >> 11) * (1.0 / 9007199254740992.0) * (double)n) % (unsigned long long)n);
  };
  auto centre_of = [&](int i) {
    const uint32_t v = vec[vq_slot(i)];
    return make_float2(h2f_bits(v & 0xFFFFu), h2f_bits(v >> 16));
  };
  if (tid == 0) sh.draw[0] = rng.next();
  __syncthreads();
  // ---- k-means++ seeding (unweighted): first centre uniform, the others with probability
  // proportional to the squared distance to the nearest centre chosen so far
  float dist[kVqPerThread];
  {
    const float2 c = centre_of(below(sh.draw[0]));
    if (tid == 0) { sh.cx[0] = (double)c.x; sh.cy[0] = (double)c.y; }
#pragma unroll
    for (int k = 0; k < kVqPerThread; ++k) {
      const uint32_t v = vec[vq_slot(base + k)];
      dist[k] = d2f(h2f_bits(v & 0xFFFFu), h2f_bits(v >> 16), c);
    }
  }
  for (int e = 1; e < E; ++e) {
    const int par = e & 1;
    if (tid == 0) { sh.draw[par] = rng.next(); sh.pick[par] = n - 1; }
    __syncthreads();
    const uint64_t r = sh.draw[par];
    const float u01 = (float)((double)(r >> 11) * (1.0 / 9007199254740992.0));
    const float total = block_scan_pick(sh, dist, n_mine, base, u01, &sh.pick[par]);
    const int pick = total > 0.f ? sh.pick[par] : below(r);
    const float2 c = centre_of(pick);
    if (tid == 0) { sh.cx[e] = (double)c.x; sh.cy[e] = (double)c.y; }
#pragma unroll
    for (int k = 0; k < kVqPerThread; ++k) {
      const uint32_t v = vec[vq_slot(base + k)];
      dist[k] = fminf(dist[k], d2f(h2f_bits(v & 0xFFFFu), h2f_bits(v >> 16), c));
    }
  }
  __syncthreads();
  // ---- Lloyd iterations
  for (int it = 0; it < a.iters; ++it) {
    for (int e = tid; e < E; e += kVqThreads) {
      sh.cf[e] = make_float2((float)sh.cx[e], (float)sh.cy[e]);
      sh.sx[e] = 0ull; sh.sy[e] = 0ull; sh.cnt[e] = 0u;
    }
    __syncthreads();
    for (int k0 = 0; k0 < n_mine; k0 += 4) {
      float x[4], y[4], wx[4], wy[4], best[4];
      int bi[4];
      uint32_t bits[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = base + k0 + q;
        bits[q] = vec[vq_slot(min(i, kVqMaxVec - 1))];
        x[q] = h2f_bits(bits[q] & 0xFFFFu); y[q] = h2f_bits(bits[q] >> 16);
        wx[q] = wy[q] = 1.f;
        if (weighted && k0 + q < n_mine) {
          const float2 wv = __ldg(reinterpret_cast<const float2*>(a.elem_w) + i);
          wx[q] = wv.x; wy[q] = wv.y;
        }
        best[q] = INFINITY; bi[q] = 0;
      }
      for (int e = 0; e < E; ++e) {
        const float2 c = sh.cf[e];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float dx = x[q] - c.x, dy = y[q] - c.y;
          const float d = weighted ? fmaf(wx[q], dx * dx, wy[q] * (dy * dy)) : fmaf(dx, dx, dy * dy);
          if (d < best[q]) { best[q] = d; bi[q] = e; }
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (k0 + q < n_mine) {
          if (weighted) {
            idx[base + k0 + q] = (uint8_t)bi[q];
          } else {
            atomicAdd(&sh.sx[bi[q]], (unsigned long long)half_fixed(bits[q] & 0xFFFFu));
            atomicAdd(&sh.sy[bi[q]], (unsigned long long)half_fixed(bits[q] >> 16));
            atomicAdd(&sh.cnt[bi[q]], 1u);
          }
        }
      }
    }
    __syncthreads();
    for (int e = tid; e < E; e += kVqThreads) {
      if (!weighted) {
        if (sh.cnt[e]) {
          sh.cx[e] = (double)(long long)sh.sx[e] * (1.0 / 16777216.0) / (double)sh.cnt[e];
          sh.cy[e] = (double)(long long)sh.sy[e] * (1.0 / 16777216.0) / (double)sh.cnt[e];
        }
      } else {
        // weighted means of Eq. 19, per dimension, members taken in vector order
        double nx = 0.0, dxs = 0.0, ny = 0.0, dys = 0.0;
        for (int i = 0; i < n; ++i) {
          if (idx[i] == (uint8_t)e) {
            const uint32_t v = vec[vq_slot(i)];
            const float2 wv = __ldg(reinterpret_cast<const float2*>(a.elem_w) + i);
            nx += (double)wv.x * (double)h2f_bits(v & 0xFFFFu); dxs += (double)wv.x;
            ny += (double)wv.y * (double)h2f_bits(v >> 16);     dys += (double)wv.y;
          }
        }
        if (dxs > 0.0) sh.cx[e] = nx / dxs;
        if (dys > 0.0) sh.cy[e] = ny / dys;
      }
    }
    __syncthreads();
  }
  // ---- centres to fp16; final assignment against the rounded centres in fp64 (exact differences,
  // products and sum each rounded once, in this order; the lowest index wins ties)
  uint32_t* aux = a.aux + (size_t)tile * E;
  for (int e = tid; e < E; e += kVqThreads) {
    const __half hx = __double2half(sh.cx[e]), hy = __double2half(sh.cy[e]);
    sh.cx[e] = (double)__half2float(hx); sh.cy[e] = (double)__half2float(hy);
    aux[e] = (uint32_t)__half_as_ushort(hx) | ((uint32_t)__half_as_ushort(hy) << 16);
  }
  __syncthreads();
  for (int k = 0; k < n_mine; ++k) {
    const int i = base + k;
    const uint32_t v = vec[vq_slot(i)];
    const double x = (double)h2f_bits(v & 0xFFFFu), y = (double)h2f_bits(v >> 16);
    double wx = 1.0, wy = 1.0;
    if (weighted) { const float2 wv = __ldg(reinterpret_cast<const float2*>(a.elem_w) + i); wx = (double)wv.x; wy = (double)wv.y; }
    double best = INFINITY;
    int bi = 0;
    for (int e = 0; e < E; ++e) {
      const double dx = x - sh.cx[e], dy = y - sh.cy[e];
      const double d = weighted ? __dadd_rn(__dmul_rn(wx, __dmul_rn(dx, dx)), __dmul_rn(wy, __dmul_rn(dy, dy)))
                                : __dadd_rn(__dmul_rn(dx, dx), __dmul_rn(dy, dy));
      if (d < best) { best = d; bi = e; }
    }
    idx[i] = (uint8_t)bi;
  }
  __syncthreads();
  // ---- bit packing (format.h)
  const int bits = a.bits;
  if (!a.is_vector) {
    const int rec = tid >> 5, L = tid & 31, g = L >> 2, t = L & 3;
    const uint32_t rb = rwkvq_vq_record_bytes(bits);
    const int mb = tr * 2 + (rec >> 3), rt = rec & 7;
    uint8_t* out = a.payload + (((size_t)mb * a.TC + tc) * 8 + rt) * rb;
    if (bits == 6) vq_pack_lane<6>(idx, rec, g, t, L, out); else vq_pack_lane<8>(idx, rec, g, t, L, out);
  } else {
    const int n_words = (int)(((((size_t)n * bits + 7) / 8 + 15) / 16 * 16) / 4);
    for (int wi = tid; wi < n_words; wi += kVqThreads) {
      uint32_t val = 0u;
      const int lo_bit = 32 * wi;
      for (int nn = lo_bit / bits; nn < n && nn * bits < lo_bit + 32; ++nn) {
        const int shft = nn * bits - lo_bit;
        val |= shft >= 0 ? (uint32_t)idx[nn] << shft : (uint32_t)idx[nn] >> (-shft);
      }
      reinterpret_cast<uint32_t*>(a.payload)[wi] = val;
    }
  }
}

// ---- representative activation (Section 4.2) -----------------------------------------------------
//
// A block takes 32 neighbouring positions: their samples are read row by row (coalesced) into
// shared memory, then each warp handles four positions.  The order statistics that the two
// percentiles interpolate between are found by counting: v is the k-th smallest sample iff
// #{samples < v} <= k < #{samples <= v}.
struct RepArgs {
  const float* samples;
  int S, n;
  int k_lo, k_hi;          // lower order statistic of each percentile (the upper one is k + 1, capped at S - 1)
  double g_lo, g_hi;       // interpolation fractions
  float* rep;
  float* rep_sq;
};

__device__ __forceinline__ double lerp_between(double a, double b, double t) {
  const double diff = b - a;
  return t >= 0.5 ? b - diff * (1.0 - t) : a + diff * t;
}

__global__ void __launch_bounds__(256) representative_kernel(const RepArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  float* tile = reinterpret_cast<float*>(smem);      // [S][33]
  const int j0 = blockIdx.x * 32;
  const int S = a.S;
  for (int i = threadIdx.x; i < S * 32; i += 256) {
    const int s = i >> 5, c = i & 31;
    tile[s * 33 + c] = (j0 + c < a.n) ? __ldg(a.samples + (size_t)s * a.n + j0 + c) : 0.f;
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int c = warp; c < 32; c += 8) {
    if (j0 + c >= a.n) break;
    const int ks[4] = {a.k_lo, min(a.k_lo + 1, S - 1), a.k_hi, min(a.k_hi + 1, S - 1)};
    float found[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    for (int i = lane; i < S; i += 32) {
      const float v = tile[i * 33 + c];
      int lt = 0, le = 0;
      for (int s = 0; s < S; ++s) {
        const float u = tile[s * 33 + c];
        lt += u < v; le += u <= v;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (lt <= ks[q] && ks[q] < le) found[q] = v;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) found[q] = fmaxf(found[q], __shfl_xor_sync(0xFFFFFFFFu, found[q], off));
    const double lo = lerp_between((double)found[0], (double)found[1], a.g_lo);
    const double hi = lerp_between((double)found[2], (double)found[3], a.g_hi);
    double sum = 0.0;
    for (int i = lane; i < S; i += 32) sum += fmin(fmax((double)tile[i * 33 + c], lo), hi);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
    if (lane == 0) {
      const double mean = sum / (double)S;
      if (a.rep) a.rep[j0 + c] = (float)mean;
      if (a.rep_sq) a.rep_sq[j0 + c] = (float)(mean * mean);
    }
  }
}

__global__ void write_header_kernel(const rwkvq_image_header h, uint8_t* image) {
  const uint32_t* src = reinterpret_cast<const uint32_t*>(&h);
  if (threadIdx.x < RWKVQ_HEADER_BYTES / 4) reinterpret_cast<uint32_t*>(image)[threadIdx.x] = src[threadIdx.x];
}

}  // namespace
}  // namespace rwkvq

extern "C" {

size_t rwkvq_quantize_workspace_bytes(void) { return 256; }

static rwkvq_status quantize_enqueue(const void* w_dev, int oc, int ic, const rwkvq_quant_cfg* cfg, const float* elem_weight_dev,
                                     void* image_dev, size_t image_bytes, rwkvq_desc* desc_out, void* workspace_dev,
                                     size_t workspace_bytes, void* stream, bool clear_flag) {
  using namespace rwkvq;
  if (!w_dev || !cfg || !image_dev || !workspace_dev || cfg->codes_in) return RWKVQ_EINVAL;
  rwkvq_desc d;
  rwkvq_status st = rwkvq_desc_for(cfg, oc, ic, &d);
  if (st != RWKVQ_OK) return st;
  const bool is_vector = cfg->method == RWKVQ_VQ && oc == 1;
  if (elem_weight_dev && !is_vector) return RWKVQ_EINVAL;
  if (cfg->method == RWKVQ_VQ && cfg->kmeans_iters < 0) return RWKVQ_EINVAL;
  if (is_vector && ic / 2 > kVqMaxVec) return RWKVQ_EUNSUPPORTED;
  if (!aligned16(w_dev) || !aligned16(workspace_dev) || (elem_weight_dev && !aligned16(elem_weight_dev)) ||
      (reinterpret_cast<uintptr_t>(image_dev) & 255u))
    return RWKVQ_EALIGN;
  if (image_bytes < d.image_bytes || workspace_bytes < rwkvq_quantize_workspace_bytes()) return RWKVQ_ENOMEM;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* img = static_cast<uint8_t*>(image_dev);
  int* flags = static_cast<int*>(workspace_dev);
  rwkvq_image_header h;
  rwkvq_fill_header(&h, d.method, d.bits, d.oc, d.ic, d.oc_pad, d.ic_pad, d.group, d.vec_dim, d.tile, d.entries, is_vector,
                    d.image_bytes, d.stream_bytes);
  h.reserved1 = RWKVQ_IMAGE_FLAG_NO_CRC;
  cudaError_t e = cudaSuccess;
  if (clear_flag) {
    e = cudaMemsetAsync(flags, 0, sizeof(int), s);
    if (e != cudaSuccess) return cuda_status(e);
  }
  write_header_kernel<<<1, 64, 0, s>>>(h, img);
  if (d.method == RWKVQ_SQ) {
    const int MB = d.oc_pad / 128, KT = d.ic_pad / 256;
    sq_quantize_kernel<<<MB * KT, 256, 0, s>>>(static_cast<const uint16_t*>(w_dev), oc, ic, KT, img + h.off_payload, flags);
  } else {
    const size_t smem = (size_t)kVqMaxVec * 5 + sizeof(VqShared);
    e = cudaFuncSetAttribute(vq_kmeans_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_status(e);
    VqArgs a;
    a.w = static_cast<const uint16_t*>(w_dev);
    a.elem_w = elem_weight_dev;
    a.ic = ic;
    a.TC = is_vector ? 1 : ic / 256;
    a.n_vec = is_vector ? ic / 2 : kVqMaxVec;
    a.bits = d.bits; a.E = d.entries; a.iters = cfg->kmeans_iters;
    a.is_vector = is_vector ? 1 : 0;
    a.seed = cfg->seed;
    a.payload = img + h.off_payload;
    a.aux = reinterpret_cast<uint32_t*>(img + h.off_aux);
    a.flags = flags;
    const int grid = is_vector ? 1 : (oc / 256) * (ic / 256);
    vq_kmeans_kernel<<<grid, kVqThreads, smem, s>>>(a);
    const size_t used = h.off_aux + h.aux_bytes;
    if (used < d.image_bytes) {
      e = cudaMemsetAsync(img + used, 0, d.image_bytes - used, s);
      if (e != cudaSuccess) return cuda_status(e);
    }
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_status(e);
  if (desc_out) *desc_out = d;
  return RWKVQ_OK;
}

rwkvq_status rwkvq_quantize_check(void* workspace_dev, void* stream) {
  using namespace rwkvq;
  if (!workspace_dev) return RWKVQ_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int host_flags = 0;
  cudaError_t e = cudaMemcpyAsync(&host_flags, workspace_dev, sizeof(int), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(workspace_dev, 0, sizeof(int), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_status(e);
  return (host_flags & kFlagNonFinite) ? RWKVQ_ENONFINITE : RWKVQ_OK;
}

rwkvq_status rwkvq_quantize_dev_async(const void* w_dev, int oc, int ic, const rwkvq_quant_cfg* cfg, const float* elem_weight_dev,
                                      void* image_dev, size_t image_bytes, rwkvq_desc* desc_out, void* workspace_dev,
                                      size_t workspace_bytes, void* stream) {
  return quantize_enqueue(w_dev, oc, ic, cfg, elem_weight_dev, image_dev, image_bytes, desc_out, workspace_dev,
                          workspace_bytes, stream, false);
}

rwkvq_status rwkvq_quantize_dev(const void* w_dev, int oc, int ic, const rwkvq_quant_cfg* cfg, const float* elem_weight_dev,
                                void* image_dev, size_t image_bytes, rwkvq_desc* desc_out, void* workspace_dev,
                                size_t workspace_bytes, void* stream) {
  rwkvq_status st = quantize_enqueue(w_dev, oc, ic, cfg, elem_weight_dev, image_dev, image_bytes, desc_out, workspace_dev,
                                     workspace_bytes, stream, true);
  if (st != RWKVQ_OK) return st;
  return rwkvq_quantize_check(workspace_dev, stream);
}

rwkvq_status rwkvq_calib_representative(const float* samples_dev, int n_samples, int n, double pct, float* rep_dev,
                                        float* rep_sq_dev, void* stream) {
  using namespace rwkvq;
  if (!samples_dev || n <= 0 || n_samples < 2 || n_samples > 1024 || !(pct >= 0.0) || !(pct < 50.0)) return RWKVQ_EINVAL;
  if (!rep_dev && !rep_sq_dev) return RWKVQ_EINVAL;
  RepArgs a;
  a.samples = samples_dev; a.S = n_samples; a.n = n; a.rep = rep_dev; a.rep_sq = rep_sq_dev;
  // percentile p of S sorted samples: position (S - 1) * p / 100, linear interpolation between neighbours
  const double v_lo = (double)(n_samples - 1) * (pct / 100.0);
  const double v_hi = (double)(n_samples - 1) * ((100.0 - pct) / 100.0);
  a.k_lo = (int)v_lo; a.g_lo = v_lo - (double)a.k_lo;
  a.k_hi = (int)v_hi; a.g_hi = v_hi - (double)a.k_hi;
  if (a.k_hi > n_samples - 1) { a.k_hi = n_samples - 1; a.g_hi = 0.0; }
  const size_t smem = (size_t)n_samples * 33 * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(representative_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return cuda_status(e);
  representative_kernel<<<(n + 31) / 32, 256, smem, static_cast<cudaStream_t>(stream)>>>(a);
  return cuda_status(cudaGetLastError());
}

}  // extern "C"
