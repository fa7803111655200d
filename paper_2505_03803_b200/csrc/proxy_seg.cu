// Coarse-to-fine proxy (Section 4.1) at finer granularity and for other input types.
//
// The paper evaluates the proxy per weight matrix and names finer granularity as future work; its
// inputs are the model's weights, whatever their type.  Two routes besides the fp16 histogram of
// proxy.cu:
//   * segments -- every seg_rows x seg_cols tile of a matrix (one output channel = a 1 x ic tile,
//     one block = e.g. 256 x 256) is sorted by ONE thread block in shared memory (bitonic network
//     on order-preserving integer keys: the sort of Eq. 5 literally), and the gaps between
//     neighbours are reduced in fp64 in a fixed order (Eqs. 6-17);
//   * a whole fp32 matrix too large for shared memory is sorted by the radix sort of the CUDA
//     toolkit's CUB (a library primitive for the sort of Eq. 5), then the same gap reduction runs over
//     the sorted array in two fixed-order passes.
// Formulas as in proxy.cu: n gaps (n = count - 1), R = sum of gaps, g' = gap / R,
//   P_c = ln n + sum g' ln g'  (0 ln 0 := 0),   t = n g' - 1,
//   P_f = sum_{k=2..K} | sum t^k / n | / (k (k-1)).
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <cub/device/device_radix_sort.cuh>
#include <vector>

#include "../../include/rwkvq.h"
#include "host_util.h"

namespace rwkvq {
namespace pseg {

constexpr int kThreads = 1024;
constexpr uint32_t kSmemKeysBytes = 131072;        // 65 536 16-bit keys or 32 768 32-bit keys
constexpr int kMaxK = 8;

struct SegResult {
  double pc, pf;
  unsigned count;
  int nonfinite;
};

// Order-preserving keys.  16-bit types are sign-magnitude: key = 0x8000 -/+ magnitude (+0 and -0
// share 0x8000).  fp32: flip all bits of negatives, the sign bit of the others.
__device__ __forceinline__ uint16_t key16(uint16_t bits) {
  const uint16_t mag = bits & 0x7FFFu;
  return (bits & 0x8000u) ? (uint16_t)(0x8000u - mag) : (uint16_t)(0x8000u + mag);
}
__device__ __forceinline__ uint16_t bits_of_key16(uint16_t key) {
  return key >= 0x8000u ? (uint16_t)(key - 0x8000u) : (uint16_t)(0x8000u | (0x8000u - key));
}
__device__ __forceinline__ uint32_t key32(uint32_t bits) { return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u); }
__device__ __forceinline__ uint32_t bits_of_key32(uint32_t key) { return (key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key; }

template <int DTYPE> struct Traits;
template <> struct Traits<RWKVQ_F16> {
  using Key = uint16_t; using Elem = uint16_t;
  static constexpr Key kPad = 0xFFFFu;
  static __device__ __forceinline__ bool finite(Elem b) { return (b & 0x7C00u) != 0x7C00u; }
  static __device__ __forceinline__ Key key(Elem b) { return key16(b); }
  static __device__ __forceinline__ double value(Key k) { return (double)__half2float(__ushort_as_half(bits_of_key16(k))); }
};
template <> struct Traits<RWKVQ_BF16> {
  using Key = uint16_t; using Elem = uint16_t;
  static constexpr Key kPad = 0xFFFFu;
  static __device__ __forceinline__ bool finite(Elem b) { return (b & 0x7F80u) != 0x7F80u; }
  static __device__ __forceinline__ Key key(Elem b) { return key16(b); }
  static __device__ __forceinline__ double value(Key k) { return (double)__uint_as_float((uint32_t)bits_of_key16(k) << 16); }
};
template <> struct Traits<RWKVQ_F32> {
  using Key = uint32_t; using Elem = uint32_t;
  static constexpr Key kPad = 0xFFFFFFFFu;
  static __device__ __forceinline__ bool finite(Elem b) { return (b & 0x7F800000u) != 0x7F800000u; }
  static __device__ __forceinline__ Key key(Elem b) { return key32(b); }
  static __device__ __forceinline__ double value(Key k) { return (double)__uint_as_float(bits_of_key32(k)); }
};

// Block-wide sum in a fixed shape (deterministic); every thread gets the total.
__device__ __forceinline__ double block_sum(double v, double* red) {
  __syncthreads();
  red[threadIdx.x] = v;
  __syncthreads();
  for (int s = kThreads / 2; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  return red[0];
}

// Terms of one gap (the difference of two neighbouring sorted values, already divided by R).
__device__ __forceinline__ void gap_terms(double gp, double n, int K, double (&acc)[kMaxK]) {
  if (gp > 0.0) acc[0] += gp * log(gp);
  const double t = n * gp - 1.0;
  double pw = t;
  for (int k = 2; k <= K; ++k) { pw *= t; acc[k - 1] += pw; }
}
__device__ __forceinline__ void finish(const double (&tot)[kMaxK], double n, int K, SegResult* res) {
  double pf = 0.0;
  for (int k = 2; k <= K; ++k) pf += fabs(tot[k - 1] / n) / (double)(k * (k - 1));
  res->pc = log(n) + tot[0];
  res->pf = pf;
}

// One block per segment: tile (blockIdx.y, blockIdx.x) of seg_rows x seg_cols elements, ragged at the
// right and bottom edges.  np2 = the power of two the padded key array has (>= the largest segment).
template <int DTYPE>
__global__ void __launch_bounds__(kThreads, 1) proxy_segment_kernel(const void* w, int oc, int ic, int seg_rows, int seg_cols,
                                                                  int np2, int K, SegResult* out) {
  using T = Traits<DTYPE>;
  using Key = typename T::Key;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  Key* keys = reinterpret_cast<Key*>(smem_raw);
  __shared__ double red[kThreads];
  __shared__ int s_bad;
  const int r0 = blockIdx.y * seg_rows, c0 = blockIdx.x * seg_cols;
  const int nr = min(seg_rows, oc - r0), nc = min(seg_cols, ic - c0);
  const int count = nr * nc;
  SegResult* res = out + (size_t)blockIdx.y * gridDim.x + blockIdx.x;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  const typename T::Elem* src = static_cast<const typename T::Elem*>(w);
  int bad = 0;
  for (int i = threadIdx.x; i < np2; i += kThreads) {
    Key k = T::kPad;
    if (i < count) {
      const typename T::Elem b = src[(size_t)(r0 + i / nc) * ic + c0 + i % nc];
      if (!T::finite(b)) bad = 1; else k = T::key(b);
    }
    keys[i] = k;
  }
  if (bad) s_bad = 1;
  __syncthreads();
  if (s_bad) {
    if (threadIdx.x == 0) { res->pc = INFINITY; res->pf = INFINITY; res->count = (unsigned)count; res->nonfinite = 1; }
    return;
  }
  // bitonic sorting network, ascending; the padding keys are the largest and end up behind the data
  for (int size = 2; size <= np2; size <<= 1)
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int p = threadIdx.x; p < np2 / 2; p += kThreads) {
        const int lo = 2 * p - (p & (stride - 1));          // index with the `stride` bit clear
        const int hi = lo + stride;
        const bool up = (lo & size) == 0;
        const Key a = keys[lo], b = keys[hi];
        if ((a > b) == up) { keys[lo] = b; keys[hi] = a; }
      }
      __syncthreads();
    }
  if (count < 2) {
    if (threadIdx.x == 0) { res->pc = INFINITY; res->pf = INFINITY; res->count = (unsigned)count; res->nonfinite = 0; }
    return;
  }
  const double vmin = T::value(keys[0]), vmax = T::value(keys[count - 1]);
  const double R = vmax - vmin, n = (double)(count - 1);
  if (!(R > 0.0)) {     // constant segment: G' is undefined
    if (threadIdx.x == 0) { res->pc = INFINITY; res->pf = INFINITY; res->count = (unsigned)count; res->nonfinite = 0; }
    return;
  }
  double acc[kMaxK];
#pragma unroll
  for (int i = 0; i < kMaxK; ++i) acc[i] = 0.0;
  for (int i = threadIdx.x; i + 1 < count; i += kThreads)
    gap_terms((T::value(keys[i + 1]) - T::value(keys[i])) / R, n, K, acc);
  double tot[kMaxK];
  for (int i = 0; i < kMaxK; ++i) tot[i] = (i == 0 || i < K) ? block_sum(acc[i], red) : 0.0;
  if (threadIdx.x == 0) { finish(tot, n, K, res); res->count = (unsigned)count; res->nonfinite = 0; }
}

// ---- whole fp32 matrix: keys sorted by the library's radix sort, then two fixed-order passes ----
__global__ void __launch_bounds__(256) f32_keys_kernel(const uint32_t* w, unsigned long long count, uint32_t* keys, int* nonfinite) {
  int bad = 0;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < count;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    const uint32_t b = w[i];
    if ((b & 0x7F800000u) == 0x7F800000u) bad = 1;
    keys[i] = key32(b);
  }
  if (bad) *nonfinite = 1;
}
constexpr int kGapBlocks = 1024;      // partial sums: [kGapBlocks][kMaxK] doubles, summed in block order
__global__ void __launch_bounds__(256) f32_gap_partials_kernel(const uint32_t* sorted, unsigned long long count, int K, double* partials) {
  __shared__ double red[256];
  const double vmin = (double)__uint_as_float(bits_of_key32(sorted[0]));
  const double vmax = (double)__uint_as_float(bits_of_key32(sorted[count - 1]));
  const double R = vmax - vmin, n = (double)(count - 1);
  double acc[kMaxK];
#pragma unroll
  for (int i = 0; i < kMaxK; ++i) acc[i] = 0.0;
  if (R > 0.0) {
    const unsigned long long per = (count - 1 + kGapBlocks - 1) / kGapBlocks;
    const unsigned long long lo = (unsigned long long)blockIdx.x * per;
    const unsigned long long hi = lo + per < count - 1 ? lo + per : count - 1;
    for (unsigned long long i = lo + threadIdx.x; i < hi; i += blockDim.x) {
      const double a = (double)__uint_as_float(bits_of_key32(sorted[i])), b = (double)__uint_as_float(bits_of_key32(sorted[i + 1]));
      gap_terms((b - a) / R, n, K, acc);
    }
  }
  for (int q = 0; q < kMaxK; ++q) {
    __syncthreads();
    red[threadIdx.x] = acc[q];
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
      if ((int)threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
      __syncthreads();
    }
    if (threadIdx.x == 0) partials[(size_t)blockIdx.x * kMaxK + q] = red[0];
  }
}
__global__ void f32_gap_final_kernel(const uint32_t* sorted, unsigned long long count, int K, const double* partials,
                                     const int* nonfinite, SegResult* res) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  res->count = (unsigned)count; res->nonfinite = *nonfinite;
  const double vmin = (double)__uint_as_float(bits_of_key32(sorted[0]));
  const double vmax = (double)__uint_as_float(bits_of_key32(sorted[count - 1]));
  if (*nonfinite || count < 2 || !(vmax - vmin > 0.0)) { res->pc = INFINITY; res->pf = INFINITY; return; }
  double tot[kMaxK];
  for (int q = 0; q < kMaxK; ++q) {
    double s = 0.0;
    for (int b = 0; b < kGapBlocks; ++b) s += partials[(size_t)b * kMaxK + q];
    tot[q] = s;
  }
  finish(tot, (double)(count - 1), K, res);
}

static int next_pow2(int v) { int p = 2; while (p < v) p <<= 1; return p; }
static size_t elem_bytes(int dtype) { return dtype == RWKVQ_F32 ? 4 : 2; }

}  // namespace pseg
}  // namespace rwkvq

using namespace rwkvq;

extern "C" {

size_t rwkvq_proxy_segments_workspace_bytes(int oc, int ic, int seg_rows, int seg_cols) {
  if (oc <= 0 || ic <= 0 || seg_rows <= 0 || seg_cols <= 0) return 0;
  const size_t nseg = (size_t)((oc + seg_rows - 1) / seg_rows) * (size_t)((ic + seg_cols - 1) / seg_cols);
  return round_up_sz(nseg * sizeof(pseg::SegResult), 256);
}

rwkvq_status rwkvq_proxy_segments(const void* w, int dtype, int oc, int ic, int seg_rows, int seg_cols, int K, double tau_c,
                                  double tau_f, double* Pc, double* Pf, int* phi, void* ws, size_t ws_bytes, void* stream) {
  if (!w || !Pc || !Pf || !phi || oc <= 0 || ic <= 0 || seg_rows <= 0 || seg_cols <= 0) return RWKVQ_EINVAL;
  if (dtype != RWKVQ_F16 && dtype != RWKVQ_BF16 && dtype != RWKVQ_F32) return RWKVQ_EINVAL;
  if (K < 2 || K > pseg::kMaxK) return RWKVQ_EINVAL;
  if (seg_rows > oc) seg_rows = oc;
  if (seg_cols > ic) seg_cols = ic;
  const long long seg_elems = (long long)seg_rows * seg_cols;
  if (seg_elems > (long long)(pseg::kSmemKeysBytes / pseg::elem_bytes(dtype))) return RWKVQ_EUNSUPPORTED;
  if (!aligned16(w)) return RWKVQ_EALIGN;
  const size_t need = rwkvq_proxy_segments_workspace_bytes(oc, ic, seg_rows, seg_cols);
  if (!ws || ws_bytes < need) return RWKVQ_ENOMEM;
  if (!aligned16(ws)) return RWKVQ_EALIGN;
  const int gx = (ic + seg_cols - 1) / seg_cols, gy = (oc + seg_rows - 1) / seg_rows;
  if (gy > 65535) return RWKVQ_EUNSUPPORTED;
  const int np2 = pseg::next_pow2((int)seg_elems);
  const size_t smem = (size_t)np2 * pseg::elem_bytes(dtype);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  pseg::SegResult* res = static_cast<pseg::SegResult*>(ws);
  const void* fn = dtype == RWKVQ_F16 ? (const void*)pseg::proxy_segment_kernel<RWKVQ_F16>
                 : dtype == RWKVQ_BF16 ? (const void*)pseg::proxy_segment_kernel<RWKVQ_BF16>
                                       : (const void*)pseg::proxy_segment_kernel<RWKVQ_F32>;
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pseg::kSmemKeysBytes);
  if (e != cudaSuccess) return cuda_status(e);
  const dim3 grid((unsigned)gx, (unsigned)gy, 1);
  if (dtype == RWKVQ_F16) pseg::proxy_segment_kernel<RWKVQ_F16><<<grid, pseg::kThreads, smem, s>>>(w, oc, ic, seg_rows, seg_cols, np2, K, res);
  else if (dtype == RWKVQ_BF16) pseg::proxy_segment_kernel<RWKVQ_BF16><<<grid, pseg::kThreads, smem, s>>>(w, oc, ic, seg_rows, seg_cols, np2, K, res);
  else pseg::proxy_segment_kernel<RWKVQ_F32><<<grid, pseg::kThreads, smem, s>>>(w, oc, ic, seg_rows, seg_cols, np2, K, res);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_status(e);
  const size_t nseg = (size_t)gx * gy;
  std::vector<pseg::SegResult> host(nseg);
  e = cudaMemcpyAsync(host.data(), res, nseg * sizeof(pseg::SegResult), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_status(e);
  rwkvq_status st = RWKVQ_OK;
  for (size_t i = 0; i < nseg; ++i) {
    Pc[i] = host[i].pc; Pf[i] = host[i].pf;
    phi[i] = (host[i].pc < tau_c && host[i].pf < tau_f) ? RWKVQ_SQ : RWKVQ_VQ;   // Eq. 18, strict <
    if (host[i].nonfinite) st = RWKVQ_ENONFINITE;
  }
  return st;
}

size_t rwkvq_proxy_f32_workspace_bytes(int oc, int ic) {
  if (oc <= 0 || ic <= 0) return 0;
  const size_t n = (size_t)oc * (size_t)ic;
  size_t temp = 0;
  if (cub::DeviceRadixSort::SortKeys(nullptr, temp, (const uint32_t*)nullptr, (uint32_t*)nullptr, (long long)n) != cudaSuccess) return 0;
  return round_up_sz(n * 4, 256) * 2 + round_up_sz(temp, 256) + round_up_sz((size_t)pseg::kGapBlocks * pseg::kMaxK * 8, 256) + 512;
}

rwkvq_status rwkvq_proxy_select_f32(const void* w, int oc, int ic, int K, double tau_c, double tau_f, double* Pc, double* Pf,
                                    int* phi, void* ws, size_t ws_bytes, void* stream) {
  if (!w || !Pc || !Pf || !phi || oc <= 0 || ic <= 0) return RWKVQ_EINVAL;
  if (K < 2 || K > pseg::kMaxK) return RWKVQ_EINVAL;
  if (!aligned16(w)) return RWKVQ_EALIGN;
  const size_t need = rwkvq_proxy_f32_workspace_bytes(oc, ic);
  if (need == 0) return RWKVQ_ECUDA;
  if (!ws || ws_bytes < need) return RWKVQ_ENOMEM;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return RWKVQ_EALIGN;
  const size_t n = (size_t)oc * (size_t)ic;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* p = static_cast<uint8_t*>(ws);
  uint32_t* keys = reinterpret_cast<uint32_t*>(p); p += round_up_sz(n * 4, 256);
  uint32_t* sorted = reinterpret_cast<uint32_t*>(p); p += round_up_sz(n * 4, 256);
  size_t temp = 0;
  cub::DeviceRadixSort::SortKeys(nullptr, temp, (const uint32_t*)nullptr, (uint32_t*)nullptr, (long long)n);
  void* temp_ptr = p; p += round_up_sz(temp, 256);
  double* partials = reinterpret_cast<double*>(p); p += round_up_sz((size_t)pseg::kGapBlocks * pseg::kMaxK * 8, 256);
  int* nonfinite = reinterpret_cast<int*>(p);
  pseg::SegResult* res = reinterpret_cast<pseg::SegResult*>(p + 256);
  cudaError_t e = cudaMemsetAsync(nonfinite, 0, 512, s);
  if (e != cudaSuccess) return cuda_status(e);
  pseg::f32_keys_kernel<<<1184, 256, 0, s>>>(static_cast<const uint32_t*>(w), n, keys, nonfinite);
  e = cub::DeviceRadixSort::SortKeys(temp_ptr, temp, keys, sorted, (long long)n, 0, 32, s);
  if (e != cudaSuccess) return cuda_status(e);
  pseg::f32_gap_partials_kernel<<<pseg::kGapBlocks, 256, 0, s>>>(sorted, n, K, partials);
  pseg::f32_gap_final_kernel<<<1, 32, 0, s>>>(sorted, n, K, partials, nonfinite, res);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_status(e);
  pseg::SegResult host;
  e = cudaMemcpyAsync(&host, res, sizeof(host), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_status(e);
  *Pc = host.pc; *Pf = host.pf;
  *phi = (host.pc < tau_c && host.pf < tau_f) ? RWKVQ_SQ : RWKVQ_VQ;
  return host.nonfinite ? RWKVQ_ENONFINITE : RWKVQ_OK;
}

}  // extern "C"
