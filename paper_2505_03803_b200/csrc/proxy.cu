// Coarse-to-fine proxy (Section 4.1).  The paper sorts the flattened weights (Eq. 5) and works on
// the gaps between neighbours.  For fp16 weights the sort is a counting sort over the 65 536 bit
// patterns, so one streaming pass over the matrix (2 bytes per weight) builds a histogram and a
// second, tiny kernel walks the occupied bins in value order:
//   D distinct values v_1 < ... < v_D give D-1 positive gaps; the other n-(D-1) gaps are ties (0).
//   R = v_D - v_1 = sum of gaps;  g'_j = (v_{j+1} - v_j) / R                          (Eq. 6)
//   P_c = ln n + sum_j g'_j ln g'_j            (Eqs. 7-9, 0 ln 0 := 0, n = oc*ic - 1)
//   t_j = n g'_j - 1 (= n delta_j, Eq. 10);  ties have t = -1
//   P_f = sum_{k=2..K} | ( sum_j t_j^k + ties * (-1)^k ) / n | / (k (k-1))            (Eq. 17 with
//         v_k = n^k / (k(k-1)) folded into the moment so nothing overflows)
// The selection rule (Eq. 18) is applied on the host from the two numbers.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>

#include <algorithm>
#include <cmath>
#include <vector>

#include "../../include/rwkvq.h"
#include "host_util.h"
#include "unpack.cuh"

namespace rwkvq {

constexpr int kBins = 65536;
constexpr int kHotHalf = 24576;            // shared-memory window: |w| below fp16 pattern 0x6000 (512.0)
constexpr int kHotBins = 2 * kHotHalf;     // 192 KB of u32 counters
constexpr int kHotBase = 0x8000 - kHotHalf;

struct ProxyResult {
  double pc, pf;
  unsigned long long count;
  int distinct, nonfinite;
  int pad[2];
  double variance, cv, range, mad, ie;   // the ablation's statistics of G' (Section 5.3)
  double pad2;
};

// Order-preserving key of an fp16 bit pattern: key = 0x8000 - |bits| for negative values,
// 0x8000 + |bits| for positive ones; +0 and -0 share key 0x8000.
__device__ __forceinline__ unsigned key_of(unsigned bits) {
  const unsigned mag = bits & 0x7FFFu;
  return (bits & 0x8000u) ? 0x8000u - mag : 0x8000u + mag;
}
// bf16 != 0: the 16 bits are a bfloat16 pattern (same sign-magnitude order, other exponent width)
__device__ __forceinline__ double value_of_key(unsigned key, int bf16 = 0) {
  const unsigned short bits = key >= 0x8000u ? (unsigned short)(key - 0x8000u) : (unsigned short)(0x8000u | (0x8000u - key));
  if (bf16) return (double)__uint_as_float((unsigned)bits << 16);
  return (double)__half2float(__ushort_as_half(bits));
}

__device__ __forceinline__ void count_one(unsigned bits, unsigned* sh, unsigned* hist, int* nonfinite, unsigned expmask) {
  if ((bits & expmask) == expmask) { *nonfinite = 1; return; }
  const unsigned key = key_of(bits);
  const unsigned rel = key - (unsigned)kHotBase;
  if (rel < (unsigned)kHotBins) atomicAdd(&sh[rel], 1u);
  else atomicAdd(&hist[key], 1u);
}

__global__ void __launch_bounds__(1024, 1) proxy_hist_kernel(const __half* w, unsigned long long n, unsigned* hist, ProxyResult* res, int bf16) {
  extern __shared__ unsigned sh[];
  const unsigned expmask = bf16 ? 0x7F80u : 0x7C00u;
  for (int j = threadIdx.x; j < kHotBins; j += blockDim.x) sh[j] = 0u;
  __syncthreads();
  int bad = 0;
  const unsigned long long nvec = n / 8;
  const uint4* wv = reinterpret_cast<const uint4*>(w);
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    const uint4 v = ldg_stream(wv + i);
    const unsigned ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      count_one(ws[k] & 0xFFFFu, sh, hist, &bad, expmask);
      count_one(ws[k] >> 16, sh, hist, &bad, expmask);
    }
  }
  if (blockIdx.x == 0) {
    for (unsigned long long i = nvec * 8 + threadIdx.x; i < n; i += blockDim.x)
      count_one((unsigned)__half_as_ushort(w[i]), sh, hist, &bad, expmask);
  }
  if (bad) res->nonfinite = 1;
  __syncthreads();
  for (int j = threadIdx.x; j < kHotBins; j += blockDim.x) {
    const unsigned c = sh[j];
    if (c) atomicAdd(&hist[j + kHotBase], c);
  }
}

// One block of 1024 threads per matrix; thread t owns keys [64t, 64t+64).
__global__ void __launch_bounds__(1024, 1) proxy_reduce_kernel(const unsigned* hist_all, ProxyResult* res_all, int K, int bf16) {
  const unsigned* hist = hist_all + (size_t)blockIdx.x * kBins;
  ProxyResult* res = res_all + blockIdx.x;
  __shared__ int s_last[1024];
  __shared__ int s_first[1024];
  __shared__ unsigned long long s_cnt[1024];
  __shared__ int s_dist[1024];
  __shared__ double s_red[1024];
  const int t = threadIdx.x, k0 = t * 64;
  int first = -1, last = -1, dist = 0;
  unsigned long long cnt = 0;
  for (int k = k0; k < k0 + 64; ++k) {
    const unsigned c = hist[k];
    if (c) { if (first < 0) first = k; last = k; ++dist; cnt += c; }
  }
  s_last[t] = last; s_first[t] = first; s_cnt[t] = cnt; s_dist[t] = dist;
  __syncthreads();
  // thread 0 turns the per-thread extremes into "previous occupied key before my segment"
  if (t == 0) {
    int prev = -1, mn = -1, mx = -1, D = 0;
    unsigned long long N = 0;
    for (int i = 0; i < 1024; ++i) {
      const int l = s_last[i], f = s_first[i];
      s_last[i] = prev;                       // now: predecessor key for segment i
      if (f >= 0) { if (mn < 0) mn = f; mx = l; prev = l; }
      D += s_dist[i]; N += s_cnt[i];
    }
    s_first[0] = mn; s_first[1] = mx; s_dist[0] = D; s_cnt[0] = N;
  }
  __syncthreads();
  const int mn = s_first[0], mx = s_first[1], D = s_dist[0];
  const unsigned long long N = s_cnt[0];
  if (D < 2 || N < 2) {
    if (t == 0) {
      res->pc = INFINITY; res->pf = INFINITY; res->count = N; res->distinct = D;
      res->variance = res->cv = res->range = res->mad = res->ie = INFINITY;
    }
    return;
  }
  const double R = value_of_key((unsigned)mx, bf16) - value_of_key((unsigned)mn, bf16);
  const double n = (double)(N - 1);
  double acc[8];  // [0] = sum g' ln g', [k-1] = sum t^k for k = 2..8
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0;
  double abs_t = 0.0, gmax = 0.0, gmin = INFINITY;   // sum |t_j|, largest and smallest positive gap
  int prev = s_last[t];
  for (int k = k0; k < k0 + 64; ++k) {
    if (hist[k] == 0u) continue;
    if (prev >= 0) {
      const double gp = (value_of_key((unsigned)k, bf16) - value_of_key((unsigned)prev, bf16)) / R;
      acc[0] += gp * log(gp);
      const double tt = n * gp - 1.0;
      double pw = tt;
      for (int kk = 2; kk <= K; ++kk) { pw *= tt; acc[kk - 1] += pw; }
      abs_t += fabs(tt);
      gmax = fmax(gmax, gp);
      gmin = fmin(gmin, gp);
    }
    prev = k;
  }
  double tot[8];
  for (int i = 0; i < 8; ++i) {   // fixed-shape tree: deterministic
    __syncthreads();
    s_red[t] = acc[i];
    __syncthreads();
    for (int s = 512; s > 0; s >>= 1) {
      if (t < s) s_red[t] += s_red[t + s];
      __syncthreads();
    }
    tot[i] = s_red[0];
  }
  // three more reductions of the same shape: sum |t|, max and min positive gap
  double extra[3];
  for (int i = 0; i < 3; ++i) {
    __syncthreads();
    s_red[t] = i == 0 ? abs_t : i == 1 ? gmax : gmin;
    __syncthreads();
    for (int s = 512; s > 0; s >>= 1) {
      if (t < s) s_red[t] = i == 0 ? s_red[t] + s_red[t + s] : i == 1 ? fmax(s_red[t], s_red[t + s]) : fmin(s_red[t], s_red[t + s]);
      __syncthreads();
    }
    extra[i] = s_red[0];
  }
  if (t == 0) {
    const double ties = n - (double)(D - 1);
    // with t = n G' - 1 (ties: t = -1):  variance = sum t^2 / n^3,  mad = sum |t| / n^2
    res->variance = (tot[1] + ties) / (n * n * n);
    res->cv = sqrt(res->variance) * n;
    res->range = extra[1] - (ties > 0.0 ? 0.0 : extra[2]);
    res->mad = (extra[0] + ties) / (n * n);
    res->ie = -tot[0];
    double pf = 0.0;
    for (int kk = 2; kk <= K; ++kk) {
      const double sign = (kk & 1) ? -1.0 : 1.0;
      pf += fabs((tot[kk - 1] + ties * sign) / n) / (double)(kk * (kk - 1));
    }
    res->pc = log(n) + tot[0];
    res->pf = pf;
    res->count = N;
    res->distinct = D;
  }
}

static size_t per_matrix_bytes() { return (size_t)kBins * 4; }

}  // namespace rwkvq

using namespace rwkvq;

extern "C" {

size_t rwkvq_proxy_workspace_bytes(int n_mats) {
  if (n_mats <= 0) return 0;
  return (size_t)n_mats * per_matrix_bytes() + round_up_sz((size_t)n_mats * sizeof(ProxyResult), 256);
}

static rwkvq_status run_proxy(const void* const* w, const int* oc, const int* ic, int n_mats, int K, void* ws,
                              size_t ws_bytes, void* stream, std::vector<ProxyResult>* out, int bf16 = 0) {
  if (!w || !oc || !ic || n_mats <= 0) return RWKVQ_EINVAL;
  if (K < 2 || K > 8) return RWKVQ_EINVAL;
  if (!ws || ws_bytes < rwkvq_proxy_workspace_bytes(n_mats)) return RWKVQ_ENOMEM;
  if (!aligned16(ws)) return RWKVQ_EALIGN;
  for (int m = 0; m < n_mats; ++m) {
    if (!w[m] || oc[m] <= 0 || ic[m] <= 0) return RWKVQ_EINVAL;
    if (!aligned16(w[m])) return RWKVQ_EALIGN;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned* hist = static_cast<unsigned*>(ws);
  ProxyResult* res = reinterpret_cast<ProxyResult*>(static_cast<uint8_t*>(ws) + (size_t)n_mats * per_matrix_bytes());
  cudaError_t e = cudaMemsetAsync(ws, 0, rwkvq_proxy_workspace_bytes(n_mats), s);
  if (e != cudaSuccess) return cuda_status(e);
  const size_t smem = (size_t)kHotBins * 4;
  e = cudaFuncSetAttribute(proxy_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return cuda_status(e);
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  for (int m = 0; m < n_mats; ++m) {
    const unsigned long long n = (unsigned long long)oc[m] * (unsigned long long)ic[m];
    unsigned long long blocks = (n / 8 + 1023) / 1024;
    if (blocks < 1) blocks = 1;
    if (blocks > (unsigned long long)sms) blocks = sms;
    proxy_hist_kernel<<<(unsigned)blocks, 1024, smem, s>>>(static_cast<const __half*>(w[m]), n, hist + (size_t)m * kBins, res + m, bf16);
  }
  proxy_reduce_kernel<<<n_mats, 1024, 0, s>>>(hist, res, K, bf16);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_status(e);
  out->resize(n_mats);
  e = cudaMemcpyAsync(out->data(), res, (size_t)n_mats * sizeof(ProxyResult), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_status(e);
  for (int m = 0; m < n_mats; ++m)
    if ((*out)[m].nonfinite) return RWKVQ_ENONFINITE;
  return RWKVQ_OK;
}

rwkvq_status rwkvq_proxy_select(const void* const* w, const int* oc, const int* ic, int n_mats, int K,
                                double tau_c, double tau_f, double* Pc, double* Pf, int* phi, void* ws,
                                size_t ws_bytes, void* stream) {
  if (!Pc || !Pf || !phi) return RWKVQ_EINVAL;
  std::vector<ProxyResult> host;
  const rwkvq_status st = run_proxy(w, oc, ic, n_mats, K, ws, ws_bytes, stream, &host);
  if (st != RWKVQ_OK && st != RWKVQ_ENONFINITE) return st;
  for (int m = 0; m < n_mats; ++m) {
    Pc[m] = host[m].pc; Pf[m] = host[m].pf;
    phi[m] = (host[m].pc < tau_c && host[m].pf < tau_f) ? RWKVQ_SQ : RWKVQ_VQ;   // Eq. 18, strict <
  }
  return st;
}

rwkvq_status rwkvq_proxy_select_bf16(const void* const* w, const int* oc, const int* ic, int n_mats, int K,
                                     double tau_c, double tau_f, double* Pc, double* Pf, int* phi, void* ws,
                                     size_t ws_bytes, void* stream) {
  if (!Pc || !Pf || !phi) return RWKVQ_EINVAL;
  std::vector<ProxyResult> host;
  const rwkvq_status st = run_proxy(w, oc, ic, n_mats, K, ws, ws_bytes, stream, &host, 1);
  if (st != RWKVQ_OK && st != RWKVQ_ENONFINITE) return st;
  for (int m = 0; m < n_mats; ++m) {
    Pc[m] = host[m].pc; Pf[m] = host[m].pf;
    phi[m] = (host[m].pc < tau_c && host[m].pf < tau_f) ? RWKVQ_SQ : RWKVQ_VQ;   // Eq. 18, strict <
  }
  return st;
}

rwkvq_status rwkvq_proxy_family(const void* const* w, const int* oc, const int* ic, int n_mats, double* stats,
                                void* ws, size_t ws_bytes, void* stream) {
  if (!stats) return RWKVQ_EINVAL;
  std::vector<ProxyResult> host;
  const rwkvq_status st = run_proxy(w, oc, ic, n_mats, 2, ws, ws_bytes, stream, &host);
  if (st != RWKVQ_OK && st != RWKVQ_ENONFINITE) return st;
  for (int m = 0; m < n_mats; ++m) {
    double* o = stats + (size_t)m * 5;
    o[0] = host[m].variance; o[1] = host[m].cv; o[2] = host[m].range; o[3] = host[m].mad; o[4] = host[m].ie;
  }
  return st;
}

rwkvq_status rwkvq_tau_for_fraction(const double* values, int n, double sq_fraction, double* tau_out) {
  if (!values || !tau_out || n <= 0 || !(sq_fraction >= 0.0) || !(sq_fraction <= 1.0)) return RWKVQ_EINVAL;
  std::vector<double> v(values, values + n);
  for (double x : v) if (x != x) return RWKVQ_EINVAL;
  std::sort(v.begin(), v.end());
  const long k = lrint(sq_fraction * (double)n);
  if (k <= 0) *tau_out = -INFINITY;
  else if (k >= n) *tau_out = INFINITY;
  else *tau_out = 0.5 * (v[k - 1] + v[k]);
  return RWKVQ_OK;
}

rwkvq_status rwkvq_tau_largest_gap(const double* values, int n, double* tau_out) {
  if (!values || !tau_out || n <= 0) return RWKVQ_EINVAL;
  std::vector<double> v;
  v.reserve((size_t)n);
  for (int i = 0; i < n; ++i) {
    if (values[i] != values[i]) return RWKVQ_EINVAL;
    if (std::isfinite(values[i])) v.push_back(values[i]);
  }
  std::sort(v.begin(), v.end());
  *tau_out = INFINITY;
  if (v.size() < 2 || v.back() == v.front()) return RWKVQ_OK;
  size_t best = 0;
  double widest = -1.0;
  for (size_t i = 0; i + 1 < v.size(); ++i) {
    const double gap = v[i + 1] - v[i];
    if (gap > widest) { widest = gap; best = i; }     // the first of equally wide gaps
  }
  *tau_out = 0.5 * (v[best] + v[best + 1]);
  return RWKVQ_OK;
}

}  // extern "C"
