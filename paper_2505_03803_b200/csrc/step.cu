// A whole decode step as one persistent launch.
//
// Decode at batch 1..16 reads every packed weight once and does almost no arithmetic per byte
// (the paper's compute-to-memory argument, Section 1 and Appendix A.3), and one projection of a
// 7B-class layer is only a few microseconds of HBM time.  Launching one kernel per projection
// leaves the memory system idle between launches, so the step is ONE kernel with one CTA per SM:
//
//   * a producer thread streams packed chunks from HBM into a ring of shared-memory slots with
//     bulk asynchronous copies (cp.async.bulk + mbarrier transaction counts).  Weights never depend
//     on activations, so the stream runs ahead across products and across stage boundaries;
//   * four stager warps build the fp16 input x_mix = x + (x_prev - x) (.) mu_hat (Appendix A.1
//     Eq. 20) for the next run of chunks into one of two shared-memory buffers, after waiting on
//     the grid-wide stage barrier when the run opens a new stage;
//   * sixteen consumer warps turn records into m16n8k16 tensor-core steps (gemv_core.cuh),
//     accumulate along K in registers and add their partial sums into y with fp32 atomics.
//
// The host plans the step once: every stage's chunks are cut into units (two chunks = sixteen
// records, one per consumer warp), dealt to the CTAs in contiguous byte-balanced ranges, and
// written as a per-CTA list of 128-byte unit descriptors plus a list of input segments.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "../../include/rwkvq.h"
#include "gemv_core.cuh"
#include "host_util.h"

namespace rwkvq {

int* device_status_ptr();  // api_misc.cu
unsigned abort_epoch();     // api_misc.cu: bumped whenever rwkvq_device_status reports a failed wait

enum { UF_FLUSH = 1, UF_STAGE_END = 2, UF_NEW_XSEG = 4, UF_END_XSEG = 8, UF_SPLIT = 16 };
// bits 16..31 of a unit's flags: index of the stage barrier a UF_STAGE_END unit arrives at
enum { UFMT_SQ = 0, UFMT_VQ6 = 1, UFMT_VQ8 = 2, UFMT_EMPTY = 3 };

struct StepUnit {            // 128 bytes; the first 48 bytes are all the producer needs
  uint64_t src0, src1;       // global addresses of chunk A / chunk B (0 = absent)
  uint64_t cb_src;           // VQ: codebook of the tile
  uint32_t bytes0, bytes1;
  uint32_t cb_bytes, flags, fmt, xcol0;   // xcol0: column of the unit's first tile inside the x segment
  uint32_t row0, oc;         // first output row of chunk A; rows of the product
  uint64_t y;                // float y[B][oc]
  uint32_t xstride, gs_off;  // geometry of the x segment: bytes between batch rows, offset of the sums
  uint32_t nbp, entries;
  uint64_t zptr[4];          // float ranges to clear before this CTA arrives at the stage barrier
  uint32_t zcount[4];
};
static_assert(sizeof(StepUnit) == 128, "unit descriptor size");

struct StepXSeg {            // 64 bytes
  uint64_t x, xprev, mu, mu_aux;
  uint32_t ic, col0, ncols;
  uint16_t mu_bits, mu_entries;
  uint32_t sums, barrier, xstride;   // barrier: index + 1 of the stage barrier to pass first
  uint32_t mu_off;                   // offset of the decoded mu row inside the buffer
};
static_assert(sizeof(StepXSeg) == 64, "segment descriptor size");

constexpr int kConsumerWarps = 16, kStagerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32, kStagerThreads = kStagerWarps * 32;
constexpr int kThreads = kConsumerThreads + kStagerThreads + 32;
constexpr int kMaxSlots = 12;
constexpr uint32_t kCtrlBytes = 1024, kXBufBytes = 32768, kMuScratch = 1024;
constexpr uint32_t kSmemLimit = 232448;  // 227 KB
constexpr uint32_t kPollLimit = 1u << 24;

struct StepArgs {
  const StepUnit* units;
  const StepXSeg* xsegs;
  const uint32_t* unit_off;   // [P+1]
  const uint32_t* xseg_off;   // [P+1]
  unsigned* counter;          // stage barriers: arrivals at barrier k, summed over all runs, in counter[k]
  unsigned target;            // arrivals that open a barrier in this run: run number * CTAs (mod 2^32)
  unsigned n_ctas;
  int* status;
  int B, n_slots;
  uint32_t slot_bytes, replica_bytes;
};

// ---- mbarrier / bulk-copy wrappers ------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait by one thread: gives up (and raises the CTA-wide abort flag) after kPollLimit polls
// or when another role of this CTA has already given up.
__device__ __forceinline__ bool mbar_wait_one(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  for (uint32_t it = 0; it < kPollLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(status, (int)RWKVQ_ETIMEOUT);
  return false;
}
// Warp-collective bounded wait: lane 0 polls, the verdict is warp-uniform; on success every lane
// observes the completed phase itself so that the data the barrier guards is visible to it.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait_one(bar, parity, abort_flag, status) ? 1 : 0;
  ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
  if (ok) {
    for (uint32_t it = 0; it < (1u << 20); ++it)
      if (mbar_try_wait(bar, parity)) break;
  }
  return ok != 0;
}
// Named barrier over `nthreads` threads that also ANDs a predicate: a uniform verdict for a role.
__device__ __forceinline__ bool named_bar_and(int id, int nthreads, bool pred) {
  uint32_t r;
  asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 p, %1, 0;\n bar.red.and.pred q, %2, %3, p;\n selp.u32 %0, 1, 0, q;\n}"
               : "=r"(r) : "r"((uint32_t)pred), "r"(id), "r"(nthreads) : "memory");
  return r != 0;
}
// Packed weights are read exactly once per step: they are marked evict-first so that streaming
// them does not push the activations, the plan and the outputs out of L2.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar, uint64_t policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

struct Ctrl {
  uint64_t full[kMaxSlots], empty[kMaxSlots];
  uint64_t xfull[2], xempty[2];
  int abort_flag;
};

// ---- roles -------------------------------------------------------------------------------------

// Producer: one warp.  Four descriptors are fetched per warp-wide 16-byte load (8 lanes each) one
// batch ahead; lane 0 waits for the slot, the owning lanes copy the descriptor into the slot
// header, lane 0 arms the barrier and issues the bulk copies.
__device__ void producer_role(const StepArgs& a, uint8_t* smem, Ctrl* ctrl, uint32_t u0, uint32_t u1) {
  const int lane = threadIdx.x & 31;
  const uint4* base = reinterpret_cast<const uint4*>(a.units);
  const uint32_t n = u1 - u0;
  volatile int* abortp = &ctrl->abort_flag;
  const uint64_t policy = policy_evict_first();
  uint4 next = make_uint4(0, 0, 0, 0);
  if ((uint32_t)(lane >> 3) < n) next = __ldg(base + (size_t)(u0 + (lane >> 3)) * 8 + (lane & 7));
  uint32_t issued = 0;
  bool ok = true;
  for (uint32_t b0 = 0; b0 < n && ok; b0 += 4) {
    const uint4 cur = next;
    const uint32_t nb = b0 + 4 + (lane >> 3);
    if (nb < n) next = __ldg(base + (size_t)(u0 + nb) * 8 + (lane & 7));
    for (int k = 0; k < 4 && b0 + k < n; ++k) {
      const uint32_t i = b0 + k;
      const int slot = (int)(i % (uint32_t)a.n_slots);
      const uint32_t round = i / (uint32_t)a.n_slots;
      uint8_t* sl = smem + kCtrlBytes + (size_t)slot * a.slot_bytes;
      int good = 1;
      if (lane == 0) good = mbar_wait_one(&ctrl->empty[slot], (round & 1u) ^ 1u, abortp, a.status) ? 1 : 0;
      good = __shfl_sync(0xFFFFFFFFu, good, 0);
      if (!good) { ok = false; break; }
      if ((lane >> 3) == k) *reinterpret_cast<uint4*>(sl + (lane & 7) * 16) = cur;
      // fields for lane 0: words of the first three 16-byte pieces of descriptor k
      const uint32_t s0l = __shfl_sync(0xFFFFFFFFu, cur.x, 8 * k), s0h = __shfl_sync(0xFFFFFFFFu, cur.y, 8 * k);
      const uint32_t s1l = __shfl_sync(0xFFFFFFFFu, cur.z, 8 * k), s1h = __shfl_sync(0xFFFFFFFFu, cur.w, 8 * k);
      const uint32_t cbl = __shfl_sync(0xFFFFFFFFu, cur.x, 8 * k + 1), cbh = __shfl_sync(0xFFFFFFFFu, cur.y, 8 * k + 1);
      const uint32_t by0 = __shfl_sync(0xFFFFFFFFu, cur.z, 8 * k + 1), by1 = __shfl_sync(0xFFFFFFFFu, cur.w, 8 * k + 1);
      const uint32_t cbb = __shfl_sync(0xFFFFFFFFu, cur.x, 8 * k + 2);
      __syncwarp();
      if (lane == 0) {
        const uint32_t tx = by0 + by1 + cbb;
        uint64_t* full = &ctrl->full[slot];
        if (tx == 0) {
          mbar_arrive(full);
        } else {
          mbar_arrive_expect_tx(full, tx);
          uint8_t* data = sl + 128;
          if (by0) bulk_g2s(data, reinterpret_cast<const void*>(((uint64_t)s0h << 32) | s0l), by0, full, policy);
          if (by1) bulk_g2s(data + by0, reinterpret_cast<const void*>(((uint64_t)s1h << 32) | s1l), by1, full, policy);
          if (cbb) bulk_g2s(data + by0 + by1, reinterpret_cast<const void*>(((uint64_t)cbh << 32) | cbl), cbb, full, policy);
        }
      }
      ++issued;
    }
  }
  if (!ok && lane == 0) {
    // Gave up: do not leave the CTA while copies this thread issued may still be landing.
    const uint32_t first = issued > (uint32_t)a.n_slots ? issued - a.n_slots : 0;
    for (uint32_t i = first; i < issued; ++i) {
      const int slot = (int)(i % (uint32_t)a.n_slots);
      const uint32_t parity = (i / (uint32_t)a.n_slots) & 1u;
      for (uint32_t it = 0; it < kPollLimit; ++it)
        if (mbar_try_wait(&ctrl->full[slot], parity)) break;
    }
  }
}

// Stagers: x_mix and, for SQ, the per-group sums of the segment, into buffer (segment index & 1).
// Everything that does not depend on the previous stage -- the decoded token-shift vector mu_hat
// and the previous token's activations -- is put into shared memory BEFORE the stage barrier, so
// that only one round of vector loads of x, the mix and the sums remain behind it.
// A thread owns 8 consecutive columns (16 bytes) of one batch row; a half-warp owns one
// 128-column group, whose three sums it reduces with shuffles.
__device__ __forceinline__ uint32_t mix2(uint32_t xr, uint32_t pr, uint32_t mr) {
  const float2 xf = __half22float2(*reinterpret_cast<const __half2*>(&xr));
  const float2 pf = __half22float2(*reinterpret_cast<const __half2*>(&pr));
  const float2 mf = __half22float2(*reinterpret_cast<const __half2*>(&mr));
  const __half2 v = __floats2half2_rn(fmaf(pf.x - xf.x, mf.x, xf.x), fmaf(pf.y - xf.y, mf.y, xf.y));
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ float pair_sum(uint32_t r) {
  const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r));
  return f.x + f.y;
}

constexpr int kStageUnroll = 4;

__device__ void stager_role(const StepArgs& a, uint8_t* smem, Ctrl* ctrl, uint8_t* xbufs, uint32_t* mucb,
                            uint32_t s0, uint32_t s1) {
  const int stid = threadIdx.x - kConsumerThreads;
  const int lane = stid & 31;
  volatile int* abortp = &ctrl->abort_flag;
  for (uint32_t si = s0; si < s1; ++si) {
    const uint32_t li = si - s0;
    const int buf = (int)(li & 1u);
    const StepXSeg sg = *reinterpret_cast<const StepXSeg*>(reinterpret_cast<const uint8_t*>(a.xsegs) + (size_t)si * 64);
    bool ok = mbar_wait_warp(&ctrl->xempty[buf], ((li >> 1) & 1u) ^ 1u, abortp, a.status);
    uint8_t* xb = xbufs + (size_t)buf * kXBufBytes;
    const uint8_t* mu = reinterpret_cast<const uint8_t*>(sg.mu);
    const __half* x = reinterpret_cast<const __half*>(sg.x);
    const __half* xp = reinterpret_cast<const __half*>(sg.xprev);
    const int nvr = (int)sg.ncols >> 3;            // 16-byte vectors per batch row
    const int total = a.B * nvr;
    const int nbp = (a.B + 1) & ~1;
    uint8_t* murow = xb + sg.mu_off;
    if (ok && mu) {
      for (int e = stid; e < (int)sg.mu_entries; e += kStagerThreads) mucb[e] = __ldg(reinterpret_cast<const uint32_t*>(sg.mu_aux) + e);
      named_bar_sync(4, kStagerThreads);
      const int bits = (int)sg.mu_bits;
      const uint32_t mask = (1u << bits) - 1u;
      for (int c8 = stid; c8 < nvr; c8 += kStagerThreads) {
        const int col = (int)sg.col0 + 8 * c8;
        uint4 m = make_uint4(0u, 0u, 0u, 0u);
        if (col < (int)sg.ic) {
          // four indices = 4*bits bits starting at a byte boundary (col/2 is a multiple of 4)
          const uint32_t byte = (uint32_t)(col >> 1) * (uint32_t)bits >> 3;
          const uint32_t* w = reinterpret_cast<const uint32_t*>(mu) + (byte >> 2);
          const uint32_t sh = (byte & 3u) * 8u;
          const uint32_t lo = __ldg(w);
          const uint32_t hi = (sh + 4u * bits > 32u) ? __ldg(w + 1) : 0u;
          const uint32_t f = __funnelshift_r(lo, hi, sh);
          m.x = mucb[f & mask];
          m.y = mucb[(f >> bits) & mask];
          m.z = mucb[(f >> (2 * bits)) & mask];
          m.w = mucb[(f >> (3 * bits)) & mask];
        }
        *reinterpret_cast<uint4*>(murow + (size_t)c8 * 16) = m;
      }
      for (int v = stid; v < total; v += kStagerThreads) {
        const int b = v / nvr, c8 = v - b * nvr;
        const int col = (int)sg.col0 + 8 * c8;
        uint4 r = make_uint4(0u, 0u, 0u, 0u);
        if (col < (int)sg.ic) r = __ldg(reinterpret_cast<const uint4*>(xp + (size_t)b * sg.ic + col));
        *reinterpret_cast<uint4*>(xb + (size_t)b * sg.xstride + (size_t)c8 * 16) = r;
      }
    }
    if (ok && sg.barrier && stid == 0) {
      // grid-wide stage barrier: every CTA has finished (and published) the previous stage.  Each
      // barrier has its own arrival counter, so a CTA without work may run ahead and arrive at
      // later barriers without releasing this one early.
      uint32_t it = 0;
      while ((int)(ld_acquire_gpu(a.counter + (sg.barrier - 1u)) - a.target) < 0) {
        if (++it >= kPollLimit || *abortp) { *abortp = 1; atomicExch(a.status, (int)RWKVQ_ETIMEOUT); ok = false; break; }
      }
    }
    if (!named_bar_and(4, kStagerThreads, ok)) return;   // all stager threads leave together
    float* gs = reinterpret_cast<float*>(xb + (size_t)a.B * sg.xstride);
    for (int v0 = stid; v0 < total; v0 += kStagerThreads * kStageUnroll) {
      uint4 raw[kStageUnroll];
#pragma unroll
      for (int u = 0; u < kStageUnroll; ++u) {
        const int v = v0 + u * kStagerThreads;
        raw[u] = make_uint4(0u, 0u, 0u, 0u);
        if (v < total) {
          const int b = v / nvr, c8 = v - b * nvr;
          const int col = (int)sg.col0 + 8 * c8;
          if (col < (int)sg.ic) raw[u] = __ldcg(reinterpret_cast<const uint4*>(x + (size_t)b * sg.ic + col));
        }
      }
#pragma unroll
      for (int u = 0; u < kStageUnroll; ++u) {
        const int v = v0 + u * kStagerThreads;
        if (v >= total) break;                      // warp-uniform: total is a multiple of 32
        const int b = v / nvr, c8 = v - b * nvr;
        uint4 r = raw[u];
        uint8_t* dst = xb + (size_t)b * sg.xstride + (size_t)c8 * 16;
        if (mu) {
          const uint4 pr = *reinterpret_cast<const uint4*>(dst);          // this thread's own earlier store
          const uint4 mr = *reinterpret_cast<const uint4*>(murow + (size_t)c8 * 16);
          r.x = mix2(r.x, pr.x, mr.x); r.y = mix2(r.y, pr.y, mr.y);
          r.z = mix2(r.z, pr.z, mr.z); r.w = mix2(r.w, pr.w, mr.w);
        }
        *reinterpret_cast<uint4*>(dst) = r;
        if (sg.sums) {
          const int o = (8 * c8) & 63;
          const float pa = pair_sum(r.x) + pair_sum(r.z), pb = pair_sum(r.y) + pair_sum(r.w);
          float sx = pa + pb;
          float t0 = fmaf((float)rwkvq_sq_bias(o, 0), pa, (float)rwkvq_sq_bias(o + 2, 0) * pb);
          float t1 = fmaf((float)rwkvq_sq_bias(o, 1), pa, (float)rwkvq_sq_bias(o + 2, 1) * pb);
#pragma unroll
          for (int d = 8; d > 0; d >>= 1) {
            sx += __shfl_xor_sync(0xFFFFFFFFu, sx, d);
            t0 += __shfl_xor_sync(0xFFFFFFFFu, t0, d);
            t1 += __shfl_xor_sync(0xFFFFFFFFu, t1, d);
          }
          if ((lane & 15) == 0) {
            const int grp = c8 >> 4;
            gs[(grp * 3 + 0) * nbp + b] = sx;
            gs[(grp * 3 + 1) * nbp + b] = t0;
            gs[(grp * 3 + 2) * nbp + b] = t1;
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&ctrl->xfull[buf]);
  }
}

template <int NB>
__device__ void consumer_role(const StepArgs& a, uint8_t* smem, Ctrl* ctrl, const uint8_t* xbufs, uint8_t* replicas,
                              uint32_t unit_base, uint32_t n_units) {
  bool dead = false;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int rec = warp & 7, half = warp >> 3;
  const int g = lane >> 2, t = lane & 3;
  volatile int* abortp = &ctrl->abort_flag;
  float acc[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
  int xcur = 1;
  uint32_t xuse = 0;  // segments acquired so far
  for (uint32_t i = 0; i < n_units; ++i) {
    const int slot = (int)(i % (uint32_t)a.n_slots);
    const uint32_t round = i / (uint32_t)a.n_slots;
    // A warp that gave up keeps walking the list (named barriers and arrivals still happen, so no
    // other warp is left waiting for it) but touches neither the slots nor global memory.
    if (!dead && !mbar_wait_warp(&ctrl->full[slot], round & 1u, abortp, a.status)) dead = true;
    const uint8_t* sl = smem + kCtrlBytes + (size_t)slot * a.slot_bytes;
    const StepUnit* u = reinterpret_cast<const StepUnit*>(sl);
    uint32_t flags = u->flags, fmt = u->fmt;
    const uint32_t by0 = u->bytes0, by1 = u->bytes1;
    if (dead) {   // the header may not have landed: take the barrier-relevant bits from the plan itself
      const StepUnit* gu = a.units + unit_base + i;
      flags = gu->flags; fmt = gu->fmt;
    }
    if (flags & UF_NEW_XSEG) {
      xcur = (int)(xuse & 1u);
      if (!dead && !mbar_wait_warp(&ctrl->xfull[xcur], (xuse >> 1) & 1u, abortp, a.status)) dead = true;
      ++xuse;
    }
    const uint8_t* data = sl + 128;
    const uint8_t* xb = xbufs + (size_t)xcur * kXBufBytes;
    const uint32_t xstride = u->xstride, nbp = u->nbp;
    if (dead) {
      if (fmt == UFMT_VQ6 || fmt == UFMT_VQ8) { named_bar_sync(1, kConsumerThreads); named_bar_sync(1, kConsumerThreads); }
    } else if (fmt == UFMT_SQ) {
      const float* gs0 = reinterpret_cast<const float*>(xb + u->gs_off);
      if (!(flags & UF_SPLIT)) {
        // warp (rec, half): record `rec` of chunk `half` (chunk B = the next 256 columns)
        SqRecord r;
        r.load_shared(data + (size_t)half * by0 + (size_t)rec * RWKVQ_SQ_RECORD_BYTES, lane);
        uint32_t w[12];
        r.words(w);
        const uint32_t col = u->xcol0 + (uint32_t)half * 256u;
        const XLane xl = make_xlane(xb + (size_t)col * 2, xstride, gs0 + (size_t)(col >> 7) * 3 * nbp, nbp, a.B, lane);
        sq_record_mma<NB>(w, r.sz, xl, acc);
      } else {
        // single chunk: the two halves take one 128-column group each
        const uint8_t* rp = data + (size_t)rec * RWKVQ_SQ_RECORD_BYTES;
        uint32_t w[6];
#pragma unroll
        for (int k = 0; k < 6; ++k) {
          const int widx = 6 * half + k;
          w[k] = *reinterpret_cast<const uint32_t*>(rp + (widx >> 2) * 512 + lane * 16 + (widx & 3) * 4);
        }
        const uint4 sz = *reinterpret_cast<const uint4*>(rp + RWKVQ_SQ_CODE_BYTES + g * 16);
        const uint32_t col = u->xcol0 + (uint32_t)half * 128u;
        const XLane xl = make_xlane(xb + (size_t)col * 2, xstride, gs0 + (size_t)(col >> 7) * 3 * nbp, nbp, a.B, lane);
        sq_group_mma<NB, 0>(w, half == 0 ? sz.x : sz.y, half == 0 ? sz.z : sz.w, xl, acc);
      }
    } else if (fmt == UFMT_VQ6 || fmt == UFMT_VQ8) {
      // replicate the tile's codebook for conflict-free lookups (all consumer warps take part)
      const uint32_t E = u->entries;
      named_bar_sync(1, kConsumerThreads);          // previous unit's lookups are done
      {
        const uint32_t* cbraw = reinterpret_cast<const uint32_t*>(data + by0 + by1);
        uint32_t* rep = reinterpret_cast<uint32_t*>(replicas);
        for (uint32_t idx = threadIdx.x; idx < E * 32u; idx += kConsumerThreads) rep[idx] = cbraw[idx >> 5];
      }
      named_bar_sync(1, kConsumerThreads);
      const uint32_t* cb_lane = reinterpret_cast<const uint32_t*>(replicas) + lane;
      const XLane xl = make_xlane(xb + (size_t)u->xcol0 * 2, xstride, nullptr, nbp, a.B, lane);
      if (!(flags & UF_SPLIT)) {
        // warp (rec, half): record `rec` of chunk `half` (chunk B = the next 128 rows, same columns)
        if (fmt == UFMT_VQ6) {
          VqRecord<6> r;
          r.load_shared(data + (size_t)half * by0 + (size_t)rec * 1536, lane);
          vq_record_mma<6, NB>(r.w, cb_lane, xl, acc);
        } else {
          VqRecord<8> r;
          r.load_shared(data + (size_t)half * by0 + (size_t)rec * 2048, lane);
          vq_record_mma<8, NB>(r.w, cb_lane, xl, acc);
        }
      } else {
        if (fmt == UFMT_VQ6) {
          VqRecord<6> r;
          r.load_shared(data + (size_t)rec * 1536, lane);
          if (half == 0) vq_record_mma<6, NB, 0, 8>(r.w, cb_lane, xl, acc);
          else vq_record_mma<6, NB, 8, 16>(r.w, cb_lane, xl, acc);
        } else {
          VqRecord<8> r;
          r.load_shared(data + (size_t)rec * 2048, lane);
          if (half == 0) vq_record_mma<8, NB, 0, 8>(r.w, cb_lane, xl, acc);
          else vq_record_mma<8, NB, 8, 16>(r.w, cb_lane, xl, acc);
        }
      }
    }
    // everything this warp needs from the slot is in registers now, except flags read above
    const uint32_t oc = u->oc;
    const uint32_t row0 = u->row0 + ((fmt != UFMT_SQ && !(flags & UF_SPLIT)) ? (uint32_t)half * 128u : 0u);
    float* y = reinterpret_cast<float*>(u->y);
    uint64_t zp[4] = {0, 0, 0, 0};
    uint32_t zc[4] = {0, 0, 0, 0};
    if ((flags & UF_STAGE_END) && !dead) {
#pragma unroll
      for (int k = 0; k < 4; ++k) { zp[k] = u->zptr[k]; zc[k] = u->zcount[k]; }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&ctrl->empty[slot]);
    if ((flags & UF_FLUSH) && !dead) {
#pragma unroll
      for (int n = 0; n < NB; ++n)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t row = row0 + (uint32_t)rec * 16u + (uint32_t)g + 8u * (uint32_t)(k >> 1);
          const int b = n * 8 + 2 * t + (k & 1);
          if (b < a.B && row < oc) atomicAdd(y + (size_t)b * oc + row, acc[n][k]);
          acc[n][k] = 0.f;
        }
    }
    if (flags & UF_END_XSEG) {
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl->xempty[xcur]);
    }
    if (flags & UF_STAGE_END) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float* z = reinterpret_cast<float*>(zp[k]);
        for (uint32_t e = threadIdx.x; e < (dead ? 0u : zc[k]); e += kConsumerThreads) z[e] = 0.f;
      }
      // The named barrier orders every consumer thread's stores and reductions before thread 0's
      // fence, which is cumulative: one fence publishes the whole CTA's share of the stage.
      named_bar_sync(2, kConsumerThreads);
      if (threadIdx.x == 0) { __threadfence(); atomicAdd(a.counter + (flags >> 16), 1u); }
    }
  }
}

template <int NB>
__global__ void __launch_bounds__(kThreads, 1) step_kernel(const StepArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem);
  uint8_t* xbufs = smem + kCtrlBytes + (size_t)a.n_slots * a.slot_bytes;
  uint32_t* mucb = reinterpret_cast<uint32_t*>(xbufs + 2 * kXBufBytes);
  uint8_t* replicas = reinterpret_cast<uint8_t*>(mucb) + kMuScratch;
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.n_slots; ++s) { mbar_init(&ctrl->full[s], 1); mbar_init(&ctrl->empty[s], kConsumerWarps); }
    for (int b = 0; b < 2; ++b) { mbar_init(&ctrl->xfull[b], kStagerWarps); mbar_init(&ctrl->xempty[b], kConsumerWarps); }
    ctrl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const uint32_t u0 = a.unit_off[blockIdx.x], u1 = a.unit_off[blockIdx.x + 1];
  const uint32_t s0 = a.xseg_off[blockIdx.x], s1 = a.xseg_off[blockIdx.x + 1];
  StepArgs la = a;
  la.units = a.units;  // descriptors are indexed globally
  const int warp = threadIdx.x >> 5;
  if (warp < kConsumerWarps) {
    consumer_role<NB>(la, smem, ctrl, xbufs, replicas, u0, u1 - u0);
  } else if (warp < kConsumerWarps + kStagerWarps) {
    stager_role(la, smem, ctrl, xbufs, mucb, s0, s1);
  } else {
    producer_role(la, smem, ctrl, u0, u1);
  }
}

// ---- host planner --------------------------------------------------------------------------------

struct PlanInfo {
  int P, B, NB, n_slots;
  unsigned runs;        // launches since the counters were last zero
  unsigned abort_epoch; // value of the abort epoch when the counters were last known good
  uint32_t slot_bytes, replica_bytes, smem_bytes;
  size_t off_unit_off, off_xseg_off, off_units, off_xsegs, off_counter, total_bytes;
  uint32_t n_units, n_xsegs, n_barriers;
};

static std::mutex g_plan_mutex;
static std::unordered_map<const void*, PlanInfo> g_plans;

struct HostUnit {
  StepUnit u;
  int op, rowkey, kt, ntiles, stage;
  uint32_t bytes;
};

// Shared-memory footprint of an input segment: B rows of x_mix, the per-group sums (SQ) and one
// row of decoded mu_hat (products with a token shift).
static uint32_t xseg_mu_off(int B, int ncols, bool sums) {
  uint32_t xstride = (uint32_t)ncols * 2u + 32u;
  uint32_t nbp = (uint32_t)((B + 1) & ~1);
  uint32_t off = (uint32_t)B * xstride + (sums ? (uint32_t)(ncols / 128) * 3u * nbp * 4u : 0u);
  return (off + 15u) & ~15u;
}
static uint32_t xseg_bytes(int B, int ncols, bool sums, bool has_mu) {
  return xseg_mu_off(B, ncols, sums) + (has_mu ? (uint32_t)ncols * 2u : 0u);
}

static rwkvq_status validate_ops(const rwkvq_gemv_op* ops, int n_ops, int B) {
  if (!ops || n_ops <= 0 || B < 1 || B > 16) return RWKVQ_EINVAL;
  for (int i = 0; i < n_ops; ++i) {
    const rwkvq_gemv_op& o = ops[i];
    rwkvq_status st = check_matrix_desc(&o.W_desc);
    if (st != RWKVQ_OK) return st;
    if (o.W_desc.oc == 1) return RWKVQ_ESHAPE;
    if (!o.W_image_dev || !o.x_fp16_dev || !o.y_dev) return RWKVQ_EINVAL;
    if ((o.mu_image_dev == nullptr) != (o.xprev_fp16_dev == nullptr)) return RWKVQ_EINVAL;
    if (o.mu_image_dev) {
      st = check_vector_desc(&o.mu_desc, o.W_desc.ic);
      if (st != RWKVQ_OK) return st;
      if (!aligned16(o.mu_image_dev) || !aligned16(o.xprev_fp16_dev)) return RWKVQ_EALIGN;
    }
    if (!aligned16(o.W_image_dev) || !aligned16(o.x_fp16_dev) || !aligned16(o.y_dev)) return RWKVQ_EALIGN;
    if (o.y_dtype != RWKVQ_F32) return RWKVQ_EUNSUPPORTED;   // partial sums are added with fp32 atomics
    if (i > 0 && o.stage < ops[i - 1].stage) return RWKVQ_EINVAL;
  }
  return RWKVQ_OK;
}

// Builds the whole plan on the host.  Returns the serialized image in `out` and fills `info`.
static rwkvq_status build_plan(const rwkvq_gemv_op* ops, int n_ops, int B, int P, std::vector<uint8_t>* out, PlanInfo* info) {
  rwkvq_status st = validate_ops(ops, n_ops, B);
  if (st != RWKVQ_OK) return st;
  bool has_vq6 = false, has_vq8 = false, has_sq = false;
  for (int i = 0; i < n_ops; ++i) {
    if (ops[i].W_desc.method == RWKVQ_SQ) has_sq = true;
    else if (ops[i].W_desc.bits == 6) has_vq6 = true;
    else has_vq8 = true;
  }
  uint32_t data_max = 0;
  if (has_sq) data_max = std::max(data_max, 2u * 8u * RWKVQ_SQ_RECORD_BYTES);
  if (has_vq6) data_max = std::max(data_max, 2u * 8u * 1536u + 256u);
  if (has_vq8) data_max = std::max(data_max, 2u * 8u * 2048u + 1024u);
  info->slot_bytes = (128u + data_max + 127u) & ~127u;
  info->replica_bytes = has_vq8 ? 256u * 128u : has_vq6 ? 64u * 128u : 0u;
  const uint32_t fixed = kCtrlBytes + 2u * kXBufBytes + kMuScratch + info->replica_bytes;
  int ns = (int)((kSmemLimit - fixed) / info->slot_bytes);
  if (ns > kMaxSlots) ns = kMaxSlots;
  if (ns < 2) return RWKVQ_EUNSUPPORTED;
  info->n_slots = ns;
  info->smem_bytes = fixed + (uint32_t)ns * info->slot_bytes;
  info->P = P; info->B = B; info->NB = B <= 8 ? 1 : 2;
  const uint32_t nbp = (uint32_t)((B + 1) & ~1);

  // stages in order of appearance
  std::vector<std::pair<int, int>> stage_ranges;  // [first op, last op) per distinct stage value
  for (int i = 0; i < n_ops;) {
    int j = i;
    while (j < n_ops && ops[j].stage == ops[i].stage) ++j;
    stage_ranges.push_back({i, j});
    i = j;
  }
  const int n_stages = (int)stage_ranges.size();
  info->n_barriers = (uint32_t)n_stages + 1;
  if (info->n_barriers > 65535u) return RWKVQ_EUNSUPPORTED;

  std::vector<std::vector<HostUnit>> cta_units(P);
  auto zero_ranges_for = [&](int stage_idx, int c, std::vector<std::pair<uint64_t, uint32_t>>* ranges) {
    // CTA c's slice of the concatenated outputs of stage `stage_idx`
    ranges->clear();
    if (stage_idx >= n_stages) return;
    uint64_t total = 0;
    for (int o = stage_ranges[stage_idx].first; o < stage_ranges[stage_idx].second; ++o) total += (uint64_t)B * ops[o].W_desc.oc;
    const uint64_t lo = total * (uint64_t)c / P, hi = total * (uint64_t)(c + 1) / P;
    uint64_t base = 0;
    for (int o = stage_ranges[stage_idx].first; o < stage_ranges[stage_idx].second; ++o) {
      const uint64_t n = (uint64_t)B * ops[o].W_desc.oc;
      const uint64_t a0 = std::max(lo, base), a1 = std::min(hi, base + n);
      if (a1 > a0) ranges->push_back({(uint64_t)(uintptr_t)ops[o].y_dev + (a0 - base) * 4, (uint32_t)(a1 - a0)});
      base += n;
    }
  };
  bool too_many_ranges = false;
  auto push_stage_end = [&](int c, int next_stage_idx, int stage_tag) {
    // attach the stage end (and the clearing of the next stage's outputs) to CTA c's list: to its
    // last unit of this stage, or to an empty unit if it has none
    std::vector<std::pair<uint64_t, uint32_t>> ranges;
    zero_ranges_for(next_stage_idx, c, &ranges);
    if (ranges.size() > 4) { too_many_ranges = true; return; }
    std::vector<HostUnit>& L = cta_units[c];
    if (L.empty() || L.back().stage != stage_tag) {
      HostUnit h{};
      h.u.fmt = UFMT_EMPTY; h.stage = stage_tag; h.op = -1; h.rowkey = -1;
      L.push_back(h);
    }
    HostUnit& last = L.back();
    last.u.flags |= UF_STAGE_END | ((uint32_t)(stage_tag + 1) << 16);   // barrier 0 = the clearing pass
    for (size_t k = 0; k < ranges.size(); ++k) { last.u.zptr[k] = ranges[k].first; last.u.zcount[k] = ranges[k].second; }
  };

  // barrier #0: clear the outputs of the first stage
  for (int c = 0; c < P; ++c) push_stage_end(c, 0, -1);

  for (int s = 0; s < n_stages; ++s) {
    std::vector<HostUnit> units;
    for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) {
      const rwkvq_desc& d = ops[o].W_desc;
      const uint8_t* img = static_cast<const uint8_t*>(ops[o].W_image_dev);
      const uint8_t* payload = img + RWKVQ_HEADER_BYTES;
      const int KT = d.ic_pad / 256;
      if (d.method == RWKVQ_SQ) {
        const int MB = d.oc_pad / 128;
        const uint32_t cb = 8u * RWKVQ_SQ_RECORD_BYTES;
        for (int rb = 0; rb < MB; ++rb)
          for (int kt = 0; kt < KT; kt += 2) {
            HostUnit h{};
            h.u.fmt = UFMT_SQ;
            h.u.src0 = (uint64_t)(uintptr_t)(payload + (size_t)(rb * KT + kt) * cb);
            h.u.bytes0 = cb;
            if (kt + 1 < KT) { h.u.src1 = h.u.src0 + cb; h.u.bytes1 = cb; h.ntiles = 2; }
            else { h.u.flags |= UF_SPLIT; h.ntiles = 1; }
            h.u.row0 = (uint32_t)rb * 128u; h.u.oc = (uint32_t)d.oc; h.u.y = (uint64_t)(uintptr_t)ops[o].y_dev;
            h.op = o; h.rowkey = rb; h.kt = kt; h.stage = s; h.bytes = h.u.bytes0 + h.u.bytes1;
            units.push_back(h);
          }
      } else {
        const int TR = d.oc / 256;
        const uint32_t rbytes = rwkvq_vq_record_bytes(d.bits), cb = 8u * rbytes;
        const uint8_t* aux = img + matrix_aux_offset(&d);
        for (int tr = 0; tr < TR; ++tr)
          for (int kt = 0; kt < KT; ++kt) {
            HostUnit h{};
            h.u.fmt = d.bits == 6 ? UFMT_VQ6 : UFMT_VQ8;
            h.u.src0 = (uint64_t)(uintptr_t)(payload + (size_t)((2 * tr) * KT + kt) * cb);
            h.u.src1 = (uint64_t)(uintptr_t)(payload + (size_t)((2 * tr + 1) * KT + kt) * cb);
            h.u.bytes0 = cb; h.u.bytes1 = cb;
            h.u.cb_src = (uint64_t)(uintptr_t)(aux + (size_t)(tr * KT + kt) * d.entries * 4);
            h.u.cb_bytes = (uint32_t)d.entries * 4u; h.u.entries = (uint32_t)d.entries;
            h.u.row0 = (uint32_t)tr * 256u; h.u.oc = (uint32_t)d.oc; h.u.y = (uint64_t)(uintptr_t)ops[o].y_dev;
            h.op = o; h.rowkey = tr; h.kt = kt; h.ntiles = 1; h.stage = s;
            h.bytes = h.u.bytes0 + h.u.bytes1 + h.u.cb_bytes;
            units.push_back(h);
          }
      }
    }
    // contiguous, byte-balanced ranges: unit -> CTA by the position of its midpoint
    uint64_t total = 0;
    for (const HostUnit& h : units) total += h.bytes;
    uint64_t run = 0;
    for (const HostUnit& h : units) {
      const uint64_t mid = run + h.bytes / 2;
      int c = (int)((mid * (uint64_t)P) / (total ? total : 1));
      if (c >= P) c = P - 1;
      cta_units[c].push_back(h);
      run += h.bytes;
    }
    for (int c = 0; c < P; ++c) push_stage_end(c, s + 1, s);
  }

  // flush flags, x segments
  std::vector<uint32_t> unit_off(P + 1, 0), xseg_off(P + 1, 0);
  std::vector<StepUnit> all_units;
  std::vector<StepXSeg> all_segs;
  for (int c = 0; c < P; ++c) {
    std::vector<HostUnit>& L = cta_units[c];
    unit_off[c] = (uint32_t)all_units.size();
    xseg_off[c] = (uint32_t)all_segs.size();
    const size_t n = L.size();
    for (size_t i = 0; i < n; ++i) {
      if (L[i].u.fmt == UFMT_EMPTY) continue;
      // next real unit of the same stage
      size_t j = i + 1;
      while (j < n && L[j].u.fmt == UFMT_EMPTY && L[j].stage == L[i].stage) ++j;
      const bool same_run = j < n && L[j].u.fmt != UFMT_EMPTY && L[j].stage == L[i].stage && L[j].op == L[i].op &&
                            L[j].rowkey == L[i].rowkey;
      if (!same_run) L[i].u.flags |= UF_FLUSH;
    }
    // segments: maximal runs of real units of one product whose column span fits the buffer
    size_t i = 0;
    while (i < n) {
      if (L[i].u.fmt == UFMT_EMPTY) { ++i; continue; }
      const int op = L[i].op;
      const bool sums = ops[op].W_desc.method == RWKVQ_SQ;
      const bool has_mu = ops[op].mu_image_dev != nullptr;
      int kmin = L[i].kt, kmax = L[i].kt + L[i].ntiles;
      size_t j = i + 1, last = i;
      while (j < n) {
        if (L[j].u.fmt == UFMT_EMPTY) { if (L[j].stage != L[i].stage) break; ++j; continue; }
        if (L[j].op != op || L[j].stage != L[i].stage) break;
        const int nmin = std::min(kmin, L[j].kt), nmax = std::max(kmax, L[j].kt + L[j].ntiles);
        if (xseg_bytes(B, (nmax - nmin) * 256, sums, has_mu) > kXBufBytes) break;
        kmin = nmin; kmax = nmax; last = j; ++j;
      }
      const int ncols = (kmax - kmin) * 256;
      if (xseg_bytes(B, ncols, sums, has_mu) > kXBufBytes) return RWKVQ_EUNSUPPORTED;
      StepXSeg sg{};
      const rwkvq_gemv_op& o = ops[op];
      sg.x = (uint64_t)(uintptr_t)o.x_fp16_dev;
      sg.ic = (uint32_t)o.W_desc.ic; sg.col0 = (uint32_t)kmin * 256u; sg.ncols = (uint32_t)ncols;
      sg.sums = sums ? 1u : 0u; sg.xstride = (uint32_t)ncols * 2u + 32u;
      sg.mu_off = xseg_mu_off(B, ncols, sums);
      sg.barrier = (uint32_t)L[i].stage + 1u;   // stage s reads its inputs after barrier s
      if (o.mu_image_dev) {
        const uint8_t* m = static_cast<const uint8_t*>(o.mu_image_dev);
        sg.xprev = (uint64_t)(uintptr_t)o.xprev_fp16_dev;
        sg.mu = (uint64_t)(uintptr_t)(m + RWKVQ_HEADER_BYTES);
        sg.mu_aux = (uint64_t)(uintptr_t)(m + vector_aux_offset(&o.mu_desc));
        sg.mu_bits = (uint16_t)o.mu_desc.bits; sg.mu_entries = (uint16_t)o.mu_desc.entries;
      }
      all_segs.push_back(sg);
      bool first = true;
      for (size_t k = i; k <= last; ++k) {
        if (L[k].u.fmt == UFMT_EMPTY) continue;
        if (first) { L[k].u.flags |= UF_NEW_XSEG; first = false; }
        L[k].u.xcol0 = (uint32_t)(L[k].kt - kmin) * 256u;
        L[k].u.xstride = sg.xstride; L[k].u.gs_off = (uint32_t)B * sg.xstride; L[k].u.nbp = nbp;
      }
      L[last].u.flags |= UF_END_XSEG;
      i = last + 1;
    }
    for (size_t k = 0; k < n; ++k) all_units.push_back(L[k].u);
  }
  unit_off[P] = (uint32_t)all_units.size();
  xseg_off[P] = (uint32_t)all_segs.size();
  // A CTA's slice of a stage's outputs may touch at most four products (descriptor space).
  if (too_many_ranges) return RWKVQ_EUNSUPPORTED;

  info->n_units = (uint32_t)all_units.size();
  info->n_xsegs = (uint32_t)all_segs.size();
  size_t off = 256;
  info->off_unit_off = off; off += round_up_sz((size_t)(P + 1) * 4, 256);
  info->off_xseg_off = off; off += round_up_sz((size_t)(P + 1) * 4, 256);
  info->off_units = off; off += round_up_sz(all_units.size() * sizeof(StepUnit), 256);
  info->off_xsegs = off; off += round_up_sz(std::max<size_t>(1, all_segs.size()) * sizeof(StepXSeg), 256);
  info->off_counter = off; off += round_up_sz((size_t)info->n_barriers * 4, 256);
  info->total_bytes = off;
  if (out) {
    out->assign(off, 0);
    memcpy(out->data() + info->off_unit_off, unit_off.data(), (size_t)(P + 1) * 4);
    memcpy(out->data() + info->off_xseg_off, xseg_off.data(), (size_t)(P + 1) * 4);
    memcpy(out->data() + info->off_units, all_units.data(), all_units.size() * sizeof(StepUnit));
    if (!all_segs.empty()) memcpy(out->data() + info->off_xsegs, all_segs.data(), all_segs.size() * sizeof(StepXSeg));
  }
  return RWKVQ_OK;
}

static int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
  return sms;
}

}  // namespace rwkvq

using namespace rwkvq;

extern "C" {

size_t rwkvq_step_plan_bytes(const rwkvq_gemv_op* ops, int n_ops, int B) {
  PlanInfo info;
  if (build_plan(ops, n_ops, B, sm_count(), nullptr, &info) != RWKVQ_OK) return 0;
  return info.total_bytes;
}

rwkvq_status rwkvq_step_plan(const rwkvq_gemv_op* ops, int n_ops, int B, void* plan_dev, size_t plan_bytes, void* stream) {
  if (!plan_dev) return RWKVQ_EINVAL;
  if (!aligned16(plan_dev)) return RWKVQ_EALIGN;
  PlanInfo info;
  std::vector<uint8_t> image;
  rwkvq_status st = build_plan(ops, n_ops, B, sm_count(), &image, &info);
  if (st != RWKVQ_OK) return st;
  if (plan_bytes < info.total_bytes) return RWKVQ_ENOMEM;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(plan_dev, image.data(), image.size(), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);   // `image` is a pageable temporary
  if (e != cudaSuccess) return cuda_status(e);
  info.runs = 0;
  info.abort_epoch = abort_epoch();   // the image just copied holds zeroed counters
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  g_plans[plan_dev] = info;
  return RWKVQ_OK;
}

rwkvq_status rwkvq_step_run(const void* plan_dev, size_t plan_bytes, void* stream) {
  if (!plan_dev) return RWKVQ_EINVAL;
  PlanInfo info;
  bool clear_counters = false;
  {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    auto it = g_plans.find(plan_dev);
    if (it == g_plans.end()) return RWKVQ_EINVAL;   // not a plan written by rwkvq_step_plan in this process
    if (plan_bytes < it->second.total_bytes) return RWKVQ_ENOMEM;
    // The arrival counters only ever grow: run r opens a barrier at r * CTAs arrivals, so a launch
    // needs no clearing pass.  A run that gave up leaves them short; start over after one.
    const unsigned epoch = abort_epoch();
    if (it->second.abort_epoch != epoch) { it->second.abort_epoch = epoch; it->second.runs = 0; clear_counters = true; }
    it->second.runs += 1;
    info = it->second;
  }
  const uint8_t* p = static_cast<const uint8_t*>(plan_dev);
  StepArgs a;
  a.units = reinterpret_cast<const StepUnit*>(p + info.off_units);
  a.xsegs = reinterpret_cast<const StepXSeg*>(p + info.off_xsegs);
  a.unit_off = reinterpret_cast<const uint32_t*>(p + info.off_unit_off);
  a.xseg_off = reinterpret_cast<const uint32_t*>(p + info.off_xseg_off);
  a.counter = reinterpret_cast<unsigned*>(const_cast<uint8_t*>(p) + info.off_counter);
  a.status = device_status_ptr();
  if (!a.status) return RWKVQ_ECUDA;
  a.B = info.B; a.n_slots = info.n_slots; a.slot_bytes = info.slot_bytes; a.replica_bytes = info.replica_bytes;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  a.n_ctas = (unsigned)info.P;
  a.target = info.runs * (unsigned)info.P;
  cudaError_t e = cudaSuccess;
  if (clear_counters) {
    e = cudaMemsetAsync(a.counter, 0, round_up_sz((size_t)info.n_barriers * 4, 256), s);
    if (e != cudaSuccess) return cuda_status(e);
  }
  const void* fn = info.NB == 1 ? (const void*)step_kernel<1> : (const void*)step_kernel<2>;
  e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)info.smem_bytes);
  if (e != cudaSuccess) return cuda_status(e);
  void* params[] = {&a};
  // Cooperative launch: all CTAs must be resident at once because they meet at the stage barrier.
  e = cudaLaunchCooperativeKernel(fn, dim3(info.P), dim3(kThreads), params, info.smem_bytes, s);
  if (e != cudaSuccess) {   // this run will never arrive: have the next one clear the counters
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    auto it = g_plans.find(plan_dev);
    if (it != g_plans.end()) it->second.abort_epoch = abort_epoch() - 1u;
  }
  return cuda_status(e);
}

rwkvq_status rwkvq_step_run_host(const void* plan_dev, size_t plan_bytes, const void* act_host, void* act_dev,
                                 size_t act_bytes, const void* y_dev, void* y_host, size_t y_bytes, void* stream) {
  if ((act_bytes && (!act_host || !act_dev)) || (y_bytes && (!y_dev || !y_host))) return RWKVQ_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (act_bytes) {
    cudaError_t e = cudaMemcpyAsync(act_dev, act_host, act_bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_status(e);
  }
  rwkvq_status st = rwkvq_step_run(plan_dev, plan_bytes, stream);
  if (st != RWKVQ_OK) return st;
  if (y_bytes) {
    cudaError_t e = cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_status(e);
  }
  return RWKVQ_OK;
}

}  // extern "C"
