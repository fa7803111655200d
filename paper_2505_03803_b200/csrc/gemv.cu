// Decode products (Appendix A.1: the W.(...) products of time- and channel-mixing) over the two
// packed formats, with the token-shift mix fused into the input stage, and the dequantisation
// probe.  One launch per product; the whole-step persistent launch lives in step.cu and reuses
// the per-record routines below.
#include <cuda_runtime.h>

#include <atomic>

#include "../../include/rwkvq.h"
#include "gemv_core.cuh"
#include "host_util.h"

namespace rwkvq {

// ---------------------------------------------------------------------------------------------
// Single-product kernel.  CTA = 8 warps; block (rb, ks) covers RPC rows (128 for SQ, 256 for
// VQ) and the column tiles [ks*nkt, min(KT, (ks+1)*nkt)).  Warp w owns record w of each chunk.
// ---------------------------------------------------------------------------------------------
template <int FMT, int NB>
__global__ void __launch_bounds__(256, 2) gemv_kernel(const GemvArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int rb = blockIdx.x, ks = blockIdx.y;
  const int kt0 = ks * a.nkt, kt1 = min(a.KT, kt0 + a.nkt);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int REC = (FMT == FMT_SQ3) ? 1 : 2;
  constexpr int RPC = 128 * REC;

  SmemLayout L = smem_layout<FMT>(a.nkt, a.B, a.mu ? a.mu_entries : 0, a.entries);
  stage_input<FMT>(smem, L, a, kt0, kt1);

  float acc[REC][NB][4];
#pragma unroll
  for (int r = 0; r < REC; ++r)
#pragma unroll
    for (int n = 0; n < NB; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[r][n][i] = 0.f;

  if constexpr (FMT == FMT_SQ3) {
    const uint8_t* rec = a.payload + ((size_t)(rb * a.KT + kt0) * 8 + warp) * RWKVQ_SQ_RECORD_BYTES;
    SqRecord cur, nxt;
    cur.load(rec, lane);
    for (int kt = kt0; kt < kt1; ++kt) {
      if (kt + 1 < kt1) nxt.load(rec + (size_t)(kt + 1 - kt0) * 8 * RWKVQ_SQ_RECORD_BYTES, lane);
      uint32_t w[12];
      cur.words(w);
      const XLane xl = make_xlane(smem + (size_t)(kt - kt0) * 512, L.xstride,
                                  reinterpret_cast<const float*>(smem + L.gs_off) + (size_t)(kt - kt0) * 2 * 3 * 16, 16, a.B, lane);
      sq_record_mma<NB>(w, cur.sz, xl, acc[0]);
      cur = nxt;
    }
  } else {
    constexpr int BITS = (FMT == FMT_VQ6) ? 6 : 8;
    constexpr int RBYTES = 64 * 32 * BITS / 8;
    const int E = a.entries;
    const uint32_t* cbg = reinterpret_cast<const uint32_t*>(a.aux) + (size_t)(rb * a.KT) * E;
    stage_codebook(smem + L.cb_off, cbg + (size_t)kt0 * E, E);
    for (int kt = kt0; kt < kt1; ++kt) {
      __syncthreads();
      if (kt + 1 < kt1)
        stage_codebook(smem + L.cb_off + (size_t)((kt + 1 - kt0) & 1) * E * 128, cbg + (size_t)(kt + 1) * E, E);
      const uint32_t* cb_lane = reinterpret_cast<const uint32_t*>(smem + L.cb_off + (size_t)((kt - kt0) & 1) * E * 128) + lane;
#pragma unroll
      for (int r = 0; r < REC; ++r) {
        const uint8_t* rec = a.payload + ((size_t)((2 * rb + r) * a.KT + kt) * 8 + warp) * RBYTES;
        VqRecord<BITS> v;
        v.load(rec, lane);
        const XLane xl = make_xlane(smem + (size_t)(kt - kt0) * 512, L.xstride, nullptr, 16, a.B, lane);
        vq_record_mma<BITS, NB>(v.w, cb_lane, xl, acc[r]);
      }
    }
  }

  // ---- epilogue: direct store, or partial sums + last-arriver reduction over the K splits
  const int g = lane >> 2, t = lane & 3;
  if (a.S == 1) {
#pragma unroll
    for (int r = 0; r < REC; ++r)
#pragma unroll
      for (int n = 0; n < NB; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          int row = rb * RPC + r * 128 + warp * 16 + g + 8 * (i >> 1);
          int b = n * 8 + 2 * t + (i & 1);
          if (b < a.B && row < a.oc) store_y(a.y, a.y_dtype, (size_t)b * a.oc + row, acc[r][n][i]);
        }
    return;
  }
  float* part = a.partial + ((size_t)(ks * gridDim.x + rb) * 16) * RPC;
#pragma unroll
  for (int r = 0; r < REC; ++r)
#pragma unroll
    for (int n = 0; n < NB; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int rl = r * 128 + warp * 16 + g + 8 * (i >> 1);
        int b = n * 8 + 2 * t + (i & 1);
        if (b < a.B) part[(size_t)b * RPC + rl] = acc[r][n][i];
      }
  __threadfence();
  __syncthreads();
  __shared__ unsigned s_last;
  if (threadIdx.x == 0) s_last = (atomicAdd(&a.counters[rb], 1u) == (unsigned)(a.S - 1));
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int idx = threadIdx.x; idx < a.B * RPC; idx += blockDim.x) {
    int b = idx / RPC, rl = idx % RPC;
    float sum = 0.f;
    for (int s = 0; s < a.S; ++s)  // fixed order: the result does not depend on arrival order
      sum += __ldcg(a.partial + ((size_t)(s * gridDim.x + rb) * 16 + b) * RPC + rl);
    int row = rb * RPC + rl;
    if (row < a.oc) store_y(a.y, a.y_dtype, (size_t)b * a.oc + row, sum);
  }
  if (threadIdx.x == 0) a.counters[rb] = 0u;  // leave the workspace zero-filled for the next call
}

// ---------------------------------------------------------------------------------------------
// Dequantisation probe: one warp per record, same unpack routines as the products.
// ---------------------------------------------------------------------------------------------
// With `ref` (the fp16 matrix the image was made from) nothing is stored: each warp instead adds up
// (w - w_hat)^2 over its record in fp64 and writes the sum to sse_partial[record].
template <int FMT>
__global__ void dequant_kernel(const uint8_t* payload, const uint8_t* aux, int oc, int ic, int KT,
                               int entries, void* out, int dtype, int n_records, const __half* ref = nullptr,
                               double* sse_partial = nullptr) {
  const int lane = threadIdx.x & 31;
  const int recid = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (recid >= n_records) return;
  const int rt = recid & 7, chunk = recid >> 3;
  const int mb = chunk / KT, kt = chunk % KT;
  const int g = lane >> 2, t = lane & 3;
  const int r0 = mb * 128 + rt * 16, c0 = kt * 256;
  double sse = 0.0;
  if constexpr (FMT == FMT_SQ3) {
    SqRecord rec;
    rec.load(payload + (size_t)recid * RWKVQ_SQ_RECORD_BYTES, lane);
    uint32_t w[12];
    rec.words(w);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t r[16];
      sq_unpack_triple(w[3 * i], w[3 * i + 1], w[3 * i + 2], r);
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int m = e >> 2, R = e & 3;
        const int row = r0 + g + 8 * (R & 1);
        const int col = c0 + 64 * i + 16 * m + 4 * t + 2 * (R >> 1);
        const uint32_t szw = rec.sz_word((R & 1) * 2 + (i >> 1));
        const float s = __half2float(__ushort_as_half((unsigned short)(szw & 0xFFFF)));
        const float z = __half2float(__ushort_as_half((unsigned short)(szw >> 16)));
        const __half2 biased = *reinterpret_cast<const __half2*>(&r[e]);
        const float bias = (float)(1024 >> rwkvq_sq_pos(e));
        const float q0 = __half2float(__low2half(biased)) - bias;   // exact: integers below 2048
        const float q1 = __half2float(__high2half(biased)) - bias;
        const float v0 = __fmul_rn(s, __fsub_rn(q0, z));
        const float v1 = __fmul_rn(s, __fsub_rn(q1, z));
        if (row < oc && col < ic) {
          if (ref) {
            const float2 wv = __half22float2(*reinterpret_cast<const __half2*>(ref + (size_t)row * ic + col));
            const double d0 = (double)wv.x - (double)v0, d1 = (double)wv.y - (double)v1;
            sse += d0 * d0 + d1 * d1;
          } else {
            store_w(out, dtype, (size_t)row * ic + col, v0);
            store_w(out, dtype, (size_t)row * ic + col + 1, v1);
          }
        }
      }
    }
  } else {
    constexpr int BITS = (FMT == FMT_VQ6) ? 6 : 8;
    VqRecord<BITS> rec;
    rec.load(payload + (size_t)recid * (64 * 32 * BITS / 8), lane);
    const uint32_t* cb = reinterpret_cast<const uint32_t*>(aux) + (size_t)((mb >> 1) * KT + kt) * entries;
#pragma unroll
    for (int n = 0; n < 64; ++n) {
      const int j = n >> 2, R = n & 3;
      const int row = r0 + g + 8 * (R & 1);
      const int col = c0 + 16 * j + 4 * t + 2 * (R >> 1);
      const uint32_t v = cb[vq_index<BITS, VqRecord<BITS>::NW>(rec.w, n)];
      const __half2 h = *reinterpret_cast<const __half2*>(&v);
      if (ref) {
        const float2 wv = __half22float2(*reinterpret_cast<const __half2*>(ref + (size_t)row * ic + col));
        const double d0 = (double)wv.x - (double)__half2float(__low2half(h)), d1 = (double)wv.y - (double)__half2float(__high2half(h));
        sse += d0 * d0 + d1 * d1;
      } else {
        store_w(out, dtype, (size_t)row * ic + col, __half2float(__low2half(h)));
        store_w(out, dtype, (size_t)row * ic + col + 1, __half2float(__high2half(h)));
      }
    }
  }
  if (ref) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) sse += __shfl_xor_sync(0xFFFFFFFFu, sse, off);
    if (lane == 0) sse_partial[recid] = sse;
  }
}

// Sum of n doubles in a fixed order (one block): the result does not depend on scheduling.
__global__ void __launch_bounds__(1024) sum_fixed_kernel(const double* v, int n, double* out) {
  __shared__ double s_red[1024];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n; i += 1024) acc += v[i];
  s_red[threadIdx.x] = acc;
  __syncthreads();
  for (int s = 512; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) s_red[threadIdx.x] += s_red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = s_red[0];
}

__global__ void dequant_vector_kernel(const uint8_t* payload, const uint8_t* aux, int ic, int bits,
                                      void* out, int dtype) {
  int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= ic / 2) return;
  uint32_t v = reinterpret_cast<const uint32_t*>(aux)[vector_index(payload, p, bits)];
  const __half2 h = *reinterpret_cast<const __half2*>(&v);
  store_w(out, dtype, 2 * (size_t)p, __half2float(__low2half(h)));
  store_w(out, dtype, 2 * (size_t)p + 1, __half2float(__high2half(h)));
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
static int fmt_of(const rwkvq_desc* d) {
  if (d->method == RWKVQ_SQ) return FMT_SQ3;
  return d->bits == 6 ? FMT_VQ6 : FMT_VQ8;
}

struct GemvPlan {
  int fmt, NRB, KT, S, nkt;
  size_t smem, ws_bytes, counters_bytes;
};

static rwkvq_status plan_gemv(const rwkvq_desc* d, int B, bool has_mu, int mu_entries, GemvPlan* p) {
  if (!d || B < 1 || B > 16) return RWKVQ_EINVAL;
  if (d->oc == 1) return RWKVQ_ESHAPE;
  rwkvq_status st = check_matrix_desc(d);
  if (st != RWKVQ_OK) return st;
  p->fmt = fmt_of(d);
  const int rpc = p->fmt == FMT_SQ3 ? 128 : 256;
  p->NRB = d->oc_pad / rpc;
  p->KT = d->ic_pad / 256;
  // Enough blocks for two per SM, bounded by the shared-memory footprint of the staged input.
  int want = (2 * 148 + p->NRB - 1) / p->NRB;
  int S = want < 1 ? 1 : (want > p->KT ? p->KT : want);
  for (;; ++S) {
    int nkt = (p->KT + S - 1) / S;
    size_t sm = p->fmt == FMT_SQ3 ? smem_layout<FMT_SQ3>(nkt, B, has_mu ? mu_entries : 0, d->entries).total
              : p->fmt == FMT_VQ6 ? smem_layout<FMT_VQ6>(nkt, B, has_mu ? mu_entries : 0, d->entries).total
                                  : smem_layout<FMT_VQ8>(nkt, B, has_mu ? mu_entries : 0, d->entries).total;
    if (sm <= 96 * 1024 || S >= p->KT) { p->nkt = nkt; p->smem = sm; break; }
  }
  p->nkt = (p->KT + S - 1) / S;
  p->S = (p->KT + p->nkt - 1) / p->nkt;  // no empty splits
  p->counters_bytes = ((size_t)p->NRB * 4 + 255) / 256 * 256;
  p->ws_bytes = p->counters_bytes + (p->S > 1 ? (size_t)p->S * p->NRB * 16 * rpc * 4 : 0);
  return RWKVQ_OK;
}

template <int FMT>
static cudaError_t launch_gemv(const GemvArgs& a, const GemvPlan& p, cudaStream_t s) {
  dim3 grid(p.NRB, p.S);
  cudaError_t e;
  if (a.B <= 8) {
    e = cudaFuncSetAttribute(gemv_kernel<FMT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
    if (e != cudaSuccess) return e;
    gemv_kernel<FMT, 1><<<grid, 256, p.smem, s>>>(a);
  } else {
    e = cudaFuncSetAttribute(gemv_kernel<FMT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
    if (e != cudaSuccess) return e;
    gemv_kernel<FMT, 2><<<grid, 256, p.smem, s>>>(a);
  }
  return cudaGetLastError();
}

}  // namespace rwkvq

using namespace rwkvq;

extern "C" {

size_t rwkvq_gemv_workspace_bytes(const rwkvq_desc* d, int B) {
  GemvPlan p;
  if (plan_gemv(d, B, true, 256, &p) != RWKVQ_OK) return 0;
  return p.ws_bytes;
}

// Every argument check of the decode product, made on the host before anything is enqueued.
static rwkvq_status check_gemv_args(const rwkvq_desc* d, const void* W, const rwkvq_desc* mud, const void* mu, const void* x,
                                    const void* xprev, int B, const void* y, int y_dtype, GemvPlan* p) {
  if (!d || !W || !x || !y) return RWKVQ_EINVAL;
  if ((mu == nullptr) != (xprev == nullptr)) return RWKVQ_EINVAL;
  if (mu && !mud) return RWKVQ_EINVAL;
  if (y_dtype != RWKVQ_F32 && y_dtype != RWKVQ_F16) return RWKVQ_EINVAL;
  if (mu) {
    rwkvq_status st = check_vector_desc(mud, d->ic);
    if (st != RWKVQ_OK) return st;
  }
  rwkvq_status st = plan_gemv(d, B, mu != nullptr, mu ? mud->entries : 0, p);
  if (st != RWKVQ_OK) return st;
  if (!aligned16(W) || !aligned16(x) || !aligned16(y) || (mu && (!aligned16(mu) || !aligned16(xprev)))) return RWKVQ_EALIGN;
  return RWKVQ_OK;
}

static rwkvq_status run_gemv(const GemvPlan& p, const rwkvq_desc* d, const void* W, const rwkvq_desc* mud, const void* mu,
                             const void* x, const void* xprev, int B, void* y, int y_dtype, void* ws, void* stream) {
  GemvArgs a;
  fill_gemv_args(&a, d, W, mud, mu, x, xprev, B, y, y_dtype);
  a.KT = p.KT; a.S = p.S; a.nkt = p.nkt;
  a.counters = static_cast<unsigned*>(ws);
  a.partial = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + p.counters_bytes);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = p.fmt == FMT_SQ3 ? launch_gemv<FMT_SQ3>(a, p, s)
                : p.fmt == FMT_VQ6 ? launch_gemv<FMT_VQ6>(a, p, s)
                                   : launch_gemv<FMT_VQ8>(a, p, s);
  return cuda_status(e);
}

rwkvq_status rwkvq_gemv(const rwkvq_desc* d, const void* W, const rwkvq_desc* mud, const void* mu,
                        const void* x, const void* xprev, int B, void* y, int y_dtype, void* ws,
                        size_t ws_bytes, void* stream) {
  GemvPlan p;
  rwkvq_status st = check_gemv_args(d, W, mud, mu, x, xprev, B, y, y_dtype, &p);
  if (st != RWKVQ_OK) return st;
  if (ws && !aligned16(ws)) return RWKVQ_EALIGN;
  if (!ws || ws_bytes < p.ws_bytes) return RWKVQ_ENOMEM;
  return run_gemv(p, d, W, mud, mu, x, xprev, B, y, y_dtype, ws, stream);
}

// ---------------------------------------------------------------------------------------------
// rwkvq_gemv for callers that cannot allocate device memory: the split-K scratch lives in a
// file-scope device array.  In host code the array's name is only a handle; its device address
// is looked up once per device (with that device current) and cached.
// ---------------------------------------------------------------------------------------------
#define RWKVQ_STATIC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[RWKVQ_STATIC_SCRATCH_BYTES];
// One entry per device ordinal, written once; atomic because any host thread may make the first
// call.  The address stays valid for the life of the device's primary context: after
// cudaDeviceReset the library has to be loaded afresh (as every other device allocation).
static std::atomic<void*> g_static_scratch_addr[64];

size_t rwkvq_gemv_static_max_scratch_bytes(void) { return RWKVQ_STATIC_SCRATCH_BYTES; }

rwkvq_status rwkvq_gemv_static(const rwkvq_desc* d, const void* W, const rwkvq_desc* mud, const void* mu,
                               const void* x, const void* xprev, int B, void* y, int y_dtype, void* stream) {
  // every argument error is reported before anything reaches the stream
  GemvPlan p;
  rwkvq_status st = check_gemv_args(d, W, mud, mu, x, xprev, B, y, y_dtype, &p);
  if (st != RWKVQ_OK) return st;
  if (p.ws_bytes > RWKVQ_STATIC_SCRATCH_BYTES) return RWKVQ_ENOMEM;   // this product needs more scratch than the built-in array holds
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_status(e);
  if (dev < 0 || dev >= 64) return RWKVQ_EUNSUPPORTED;
  void* ws = g_static_scratch_addr[dev].load(std::memory_order_acquire);
  if (!ws) {
    e = cudaGetSymbolAddress(&ws, g_static_scratch);
    if (e != cudaSuccess) return cuda_status(e);
    g_static_scratch_addr[dev].store(ws, std::memory_order_release);
  }
  // The array keeps whatever the previous call left: the arrival counters must start at zero.
  e = cudaMemsetAsync(ws, 0, p.counters_bytes, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_status(e);
  return run_gemv(p, d, W, mud, mu, x, xprev, B, y, y_dtype, ws, stream);
}

rwkvq_status rwkvq_dequant(const rwkvq_desc* d, const void* W, void* out, int dtype, void* stream) {
  if (!d || !W || !out) return RWKVQ_EINVAL;
  if (dtype != RWKVQ_F32 && dtype != RWKVQ_BF16) return RWKVQ_EINVAL;
  if (!aligned16(W) || !aligned16(out)) return RWKVQ_EALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint8_t* img = static_cast<const uint8_t*>(W);
  if (d->oc == 1) {
    rwkvq_status st = check_vector_desc(d, d->ic);
    if (st != RWKVQ_OK) return st;
    int n = d->ic / 2;
    dequant_vector_kernel<<<(n + 255) / 256, 256, 0, s>>>(img + RWKVQ_HEADER_BYTES, img + vector_aux_offset(d), d->ic, d->bits, out, dtype);
    return cuda_status(cudaGetLastError());
  }
  rwkvq_status st = check_matrix_desc(d);
  if (st != RWKVQ_OK) return st;
  const int KT = d->ic_pad / 256, nrec = (d->oc_pad / 128) * KT * 8;
  const uint8_t* payload = img + RWKVQ_HEADER_BYTES;
  const uint8_t* aux = img + matrix_aux_offset(d);
  const int fmt = fmt_of(d);
  dim3 grid((nrec + 3) / 4);
  if (fmt == FMT_SQ3) dequant_kernel<FMT_SQ3><<<grid, 128, 0, s>>>(payload, aux, d->oc, d->ic, KT, d->entries, out, dtype, nrec);
  else if (fmt == FMT_VQ6) dequant_kernel<FMT_VQ6><<<grid, 128, 0, s>>>(payload, aux, d->oc, d->ic, KT, d->entries, out, dtype, nrec);
  else dequant_kernel<FMT_VQ8><<<grid, 128, 0, s>>>(payload, aux, d->oc, d->ic, KT, d->entries, out, dtype, nrec);
  return cuda_status(cudaGetLastError());
}

size_t rwkvq_quant_error_workspace_bytes(const rwkvq_desc* d) {
  if (!d || d->oc == 1 || check_matrix_desc(d) != RWKVQ_OK) return 0;
  return (size_t)(d->oc_pad / 128) * (d->ic_pad / 256) * 8 * sizeof(double) + 256;
}

rwkvq_status rwkvq_quant_error(const void* w, const rwkvq_desc* d, const void* W, double* sse_host, void* ws,
                               size_t ws_bytes, void* stream) {
  if (!w || !d || !W || !sse_host || !ws) return RWKVQ_EINVAL;
  if (d->oc == 1) return RWKVQ_ESHAPE;
  rwkvq_status st = check_matrix_desc(d);
  if (st != RWKVQ_OK) return st;
  if (!aligned16(w) || !aligned16(W) || !aligned16(ws)) return RWKVQ_EALIGN;
  if (ws_bytes < rwkvq_quant_error_workspace_bytes(d)) return RWKVQ_ENOMEM;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint8_t* img = static_cast<const uint8_t*>(W);
  const int KT = d->ic_pad / 256, nrec = (d->oc_pad / 128) * KT * 8;
  const uint8_t* payload = img + RWKVQ_HEADER_BYTES;
  const uint8_t* aux = img + matrix_aux_offset(d);
  double* total = static_cast<double*>(ws);
  double* partial = reinterpret_cast<double*>(static_cast<uint8_t*>(ws) + 256);
  const __half* ref = static_cast<const __half*>(w);
  const int fmt = fmt_of(d);
  dim3 grid((nrec + 3) / 4);
  if (fmt == FMT_SQ3) dequant_kernel<FMT_SQ3><<<grid, 128, 0, s>>>(payload, aux, d->oc, d->ic, KT, d->entries, nullptr, 0, nrec, ref, partial);
  else if (fmt == FMT_VQ6) dequant_kernel<FMT_VQ6><<<grid, 128, 0, s>>>(payload, aux, d->oc, d->ic, KT, d->entries, nullptr, 0, nrec, ref, partial);
  else dequant_kernel<FMT_VQ8><<<grid, 128, 0, s>>>(payload, aux, d->oc, d->ic, KT, d->entries, nullptr, 0, nrec, ref, partial);
  sum_fixed_kernel<<<1, 1024, 0, s>>>(partial, nrec, total);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaMemcpyAsync(sse_host, total, sizeof(double), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  return cuda_status(e);
}

}  // extern "C"
