// A whole decode step as one persistent launch.
//
// Decode at batch 1..16 reads every packed weight once and does almost no arithmetic per byte
// (the paper's compute-to-memory argument, Section 1 and Appendix A.3), and one projection of a
// 7B-class layer is only a few microseconds of HBM time.  The step is therefore ONE cooperative
// kernel with one CTA per SM, built around these ideas:
//
//   * Weights never depend on activations, so each consumer warp owns a private ring of
//     shared-memory entries that it keeps full itself with 16-byte asynchronous copies
//     (cp.async), one 16-row x 256-column record per entry, running ahead across products and
//     across stage boundaries: HBM keeps streaming while the CTAs synchronise.  A producer warp
//     (one lane per consumer warp) walks the schedule and hands each warp, a few items ahead, a
//     32-byte header per record: where it is, where its inputs are, what to do with the
//     accumulators.  All index arithmetic of the schedule stays off the consumer warps.
//   * A product's K range is cut into slabs short enough for a CTA to hold the slab's inputs in
//     shared memory (one slab at batch 1; more at larger batches).  A 16-row slice of a slab
//     belongs to ONE CTA; its records are dealt to the CTA's consumer warps in contiguous runs along
//     K.  A warp accumulates a run in registers (m16n8k16 tensor-core steps, fp32), writes one
//     partial per run to shared memory, and the last warp to finish the slice adds the partials in
//     warp order.  With one slab the sums are the output rows (plain stores); with several, every
//     CTA writes its slab's sums to a scratch area and the last CTA to arrive adds the slabs in slab
//     order.  No atomics on outputs, no clearing pass, bit-reproducible results.
//   * Inputs: every CTA mixes the slab of activations it needs itself, right after the stage
//     barrier opens (x_mix = x + (x_prev - x) (.) mu_hat, Appendix A.1 Eq. 20; x_prev and mu_hat
//     of a thread's first vectors are fetched before the barrier opens), rounds to fp16 and keeps
//     the per-group sums the factored dequantisation needs.
//   * The stage order ("every product of stage s is complete before any activation of stage s+1 is
//     read") is a flag-array grid barrier: a CTA publishes the number of stages it has completed
//     with one release store to its own word, and one auxiliary warp per CTA polls all words.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "../../include/rwkvq.h"
#include "gemv_core.cuh"
#include "host_util.h"

namespace rwkvq {

int* device_status_ptr();  // api_misc.cu
unsigned abort_epoch();     // api_misc.cu: bumped whenever rwkvq_device_status reports a failed wait

// ---- plan records shared by host and device -----------------------------------------------------

enum { DK_PHASE = 0, DK_END = 2 };
enum : uint32_t {
  DF_FIRST = 1u << 8,    // first phase of a stage for this CTA: the stage barrier is awaited before it
  DF_LAST = 1u << 9,     // last phase of the stage: the warps report the stage after it
  DF_MU = 1u << 10, DF_SUMS = 1u << 11,
  DF_SYNC = 1u << 12,    // every consumer warp must have left the earlier phases of the stage
  DF_GROUP = 1u << 13,   // first phase of a group whose inputs are staged together
  DF_GLAST = 1u << 14    // last phase of that group
};
// kind in bits 0..3, format (FMT_*) in bits 4..5 of kind_flags

// One phase of a CTA: slices [row0/16, row0/16 + S) of one product, column tiles [kt0, kt0 + T) (one
// K slab).  Item i of the S x T grid (slice-major) goes to consumer warp w with
// w*N/CW <= i < (w+1)*N/CW  (N = S*T).
struct PhaseDesc {           // 128 bytes
  uint32_t kind_flags, stage;
  uint64_t src;              // payload of the product's image
  uint64_t cb;               // VQ: codebooks of the image
  uint64_t y;                // float y[B][oc]
  uint32_t oc, row0;         // rows of the product; first row of the phase
  uint32_t S, KT;            // slices of the phase; column tiles of the product
  uint32_t T, kt0;           // tiles of the slab; its first tile
  uint32_t xoff, xstride;    // bytes: the slab's input rows inside the input area
  uint32_t gsoff, cnt_base;  // bytes: group sums; first slice counter of the phase
  uint32_t ks_part;          // slabs of the product | this slab's number << 16
  uint32_t gslot0;           // several slabs: scratch slot of (slice row0/16, slab 0); slice i: + i * slabs
  uint32_t post_value;       // stages to report complete when the phase's stage is done
  uint32_t ic;
  uint64_t x, xprev, mu, mu_aux;   // the caller's inputs
  uint16_t mu_bits, mu_entries;
  uint32_t slot_set;         // which set of partial-sum slots the phase uses (phases of one stage alternate)
};
static_assert(sizeof(PhaseDesc) == 128, "phase descriptor size");

// run header flags (word 2 of the 32-byte header the producer writes for every run; bits 0..8: records of the run,
// 9..15: slice counter, 16..23: warps that hold a part of the slice, 24..28: the first of them)
enum : uint32_t { IF_RSELF = 1u << 29, IF_RFIRST = 1u << 30 };

constexpr int kConsumerWarps = 16;   // per CTA, plus one producer and one auxiliary warp
constexpr int kMaxCW = 24, kHeaderRing = 16, kDescRing = 32, kCnt = 128;
constexpr int kMaxVals = (16 * 16 + 31) / 32;   // elements of a slice's [batch][16 rows] block per lane
constexpr uint32_t kCtrlBytes = 2048, kDescBytes = kDescRing * 128;
constexpr uint32_t kSmemLimit = 232448;  // 227 KB
constexpr uint32_t kDefaultPollLimit = 1u << 22;

struct StepArgs {
  const PhaseDesc* descs;
  const uint32_t* desc_off;   // [P+1]
  const uint32_t* init_post;  // [P] stages a CTA may report complete before it has consumed anything
  unsigned* flags;            // [P] stages completed by each CTA, summed over all runs
  unsigned base;              // value of every flag when this run starts
  int* status;
  uint32_t poll_limit;
  unsigned wait_skew;         // added to every barrier target (0; a test sets it to make the waits run out)
  int B, nbp, depth;
  uint32_t entry_bytes, slot_floats;
  uint32_t off_hq, off_partial, off_x, off_ring;
  float* gpart;               // scratch slots of slot_floats floats: a slab's sums of one slice
  unsigned* gcnt;             // per slot of slab 0: slabs of the slice that have arrived
  unsigned long long* trace;  // rwkvq_step_trace: per-warp counters, else NULL
};

// ---- small wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// The hint lets the hardware park the thread for up to that many nanoseconds (it is woken when
// the phase completes), so that waiting warps do not compete for issue slots with computing ones.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(2000u) : "memory");
  return ok != 0;
}
// Packed weights are read exactly once per step: they are marked evict-first so that streaming
// them does not push the activations, the plan and the outputs out of L2.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_gpu(unsigned* p, unsigned v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned atom_add_acq_rel_gpu(unsigned* p, unsigned v) {
  unsigned old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void fence_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
__device__ __forceinline__ uint32_t smem_add_acq_rel(uint32_t* p, uint32_t v) {
  uint32_t old;
  asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(smem_u32(p)), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ uint32_t ld_acquire_cta(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_cta(uint32_t* p, uint32_t v) {
  asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
// Named barrier over `nthreads` threads that also ANDs a predicate: a uniform verdict for a role.
__device__ __forceinline__ bool named_bar_and(int id, int nthreads, bool pred) {
  uint32_t r;
  asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 p, %1, 0;\n bar.red.and.pred q, %2, %3, p;\n selp.u32 %0, 1, 0, q;\n}"
               : "=r"(r) : "r"((uint32_t)pred), "r"(id), "r"(nthreads) : "memory");
  return r != 0;
}

struct Ctrl {
  uint64_t open;               // the aux warp arrives once per stage this CTA takes part in
  uint32_t warps_done;         // consumer warps that have left a stage, summed over the stages so far
  uint32_t hq_head[kMaxCW];    // item headers written by the producer lane of each consumer warp
  uint32_t hq_tail[kMaxCW];    // ... and read by the warp
  uint32_t desc_hi;            // descriptors copied into the ring so far
  uint32_t desc_tail;          // descriptors below this one are no longer needed by the consumer warps
  uint32_t prod_tail;          // ... nor by any lane of the producer warp
  int abort_flag;
  uint32_t cnt[kCnt];          // per-slice count of warps that have written their partial
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block");

// The CTA's dynamic shared memory.  The record loop addresses it by 32-bit offsets from this symbol.
extern __shared__ __align__(128) uint8_t smem_base[];

struct Env {
  const StepArgs& a;
  uint8_t* smem;
  Ctrl* ctrl;
  volatile int* abortp;
};

// Optional per-warp cycle accounting (rwkvq_step_trace): kTraceSlots 64-bit counters per warp,
// (CW + 2) warps per CTA.  Compiled into separate kernel instances, so the ordinary launch carries
// none of it.
constexpr int kTraceSlots = 16, kTraceStages = 64;
enum { TR_WAIT_FULL = 0, TR_WAIT_OPEN, TR_PRE, TR_POST, TR_ITEMS, TR_FLUSH, TR_NITEMS, TR_TOTAL, TR_WAIT_DESC,
       TR_P_ITER = 0, TR_P_ISSUED, TR_P_TOTAL, TR_P_IDLE, TR_P_WORK,
       TR_A_WAIT = 0, TR_A_POLLS, TR_A_REFILL, TR_A_TOTAL };
template <bool TRACE>
struct Tracer {
  unsigned long long v[TRACE ? kTraceSlots : 1];
  __device__ __forceinline__ Tracer() {
    if constexpr (TRACE) for (int k = 0; k < kTraceSlots; ++k) v[k] = 0ull;
  }
  __device__ __forceinline__ long long now() const { if constexpr (TRACE) return clock64(); else return 0; }
  __device__ __forceinline__ void add(int slot, long long t0) { if constexpr (TRACE) v[slot] += (unsigned long long)(clock64() - t0); }
  __device__ __forceinline__ void count(int slot, unsigned n = 1u) { if constexpr (TRACE) v[slot] += n; }
  // Timeline of the first kTraceStages stages of a CTA: when its last warp published the stage
  // (0), when the auxiliary warp saw the barrier open (1), when consumer warp 0 woke up (2) and when
  // the consumers had the stage's inputs staged (3); SM clock, comparable within one CTA only.
  __device__ __forceinline__ static void stamp(unsigned long long* trace, uint32_t stage, int what) {
    if constexpr (TRACE) {
      if (trace && stage < (uint32_t)kTraceStages)
        trace[(size_t)gridDim.x * (blockDim.x >> 5) * kTraceSlots + ((size_t)blockIdx.x * kTraceStages + stage) * 4 + what] = (unsigned long long)clock64();
    }
  }
  __device__ __forceinline__ void store(unsigned long long* trace) const {
    if constexpr (TRACE) {
      if (trace && (threadIdx.x & 31) == 0) {
        unsigned long long* dst = trace + ((size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * kTraceSlots;
        for (int k = 0; k < kTraceSlots; ++k) dst[k] = v[k];
      }
    }
  }
};

__device__ __forceinline__ void give_up(const Env& e) {
  *e.abortp = 1;
  atomicExch(e.a.status, (int)RWKVQ_ETIMEOUT);
}
// Bounded wait on an mbarrier phase: gives up (and raises the CTA-wide abort flag) after
// poll_limit polls or when another role of this CTA has already given up.
__device__ __forceinline__ bool mbar_wait(const Env& e, uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < e.a.poll_limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 15u) == 15u && *e.abortp) return false;
  }
  give_up(e);
  return false;
}
__device__ __forceinline__ const PhaseDesc* desc_slot(const Env& e, uint32_t p) {
  return reinterpret_cast<const PhaseDesc*>(e.smem + kCtrlBytes) + (p % (uint32_t)kDescRing);
}
// Bounded wait until descriptor p is in the ring.
__device__ __forceinline__ bool wait_desc(const Env& e, uint32_t p) {
  for (uint32_t it = 0; it < (e.a.poll_limit << 4); ++it) {
    if ((int)(ld_acquire_cta(&e.ctrl->desc_hi) - p) > 0) return true;
    if ((it & 63u) == 63u && *e.abortp) return false;
    __nanosleep(64);
  }
  give_up(e);
  return false;
}

// The share [i0, i1) of a phase's N = S*T items that consumer warp w of CW owns.
template <int CW>
__host__ __device__ __forceinline__ void item_range(uint32_t N, uint32_t w, uint32_t& i0, uint32_t& i1) {
  if (N >= (uint32_t)CW) { i0 = w * N / (uint32_t)CW; i1 = (w + 1u) * N / (uint32_t)CW; }
  else { i0 = w < N ? w : N; i1 = w + 1u < N ? w + 1u : N; }
}

// ---- producer: one lane per consumer warp ---------------------------------------------------------
//
// A RUN is the part of one slice that one consumer warp owns: consecutive column tiles of the
// slab.  Lane w walks the CTA's phases and writes, for every run of warp w in consumption order, a
// 32-byte header into warp w's header ring: where the run's first record (and, for VQ, its
// codebook) is in global memory, how many records follow at the fixed stride of a column tile,
// where the inputs of the first tile are in shared memory, and who else holds a part of the slice.
// It stays a few runs ahead of the consumer, which issues the copies itself.
//   q0 = { byte offset of the first tile's inputs in shared memory, ... of its group sums, flags | records, first row of the slice }
//   q1 = { address of the first record | format, codebook address - record address, unused }
template <int CW, bool TRACE>
__device__ void producer_role(const Env& e) {
  const StepArgs& a = e.a;
  Tracer<TRACE> tr;
  const long long t_begin = tr.now();
  const uint32_t w = threadIdx.x & 31u;
  const bool active = w < (uint32_t)CW;
  uint8_t* hq = e.smem + a.off_hq + (size_t)w * kHeaderRing * 32u;
  const uint32_t sums_tile = 2u * 3u * (uint32_t)a.nbp * 4u;   // bytes of group sums per 256-column tile
  uint32_t p = 0;              // descriptor this lane works on
  bool have = false, done = !active;
  // current phase
  uint32_t kf = 0, KT = 0, T = 0, kt0 = 0, N = 0, i0 = 0, i1 = 0, rec_bytes = 0, cb_bytes = 0;
  uint32_t xoff = 0, gsoff = 0, row0 = 0, cnt_base = 0;
  uint64_t src0 = 0, cb0 = 0;
  uint32_t i = 0, sl0 = 0;     // first item of the next run; the warp's first slice of the phase
  uint32_t n = 0;              // headers written
  uint32_t tail = 0;           // headers the consumer is known to have read
  uint32_t idle = 0, last_pmin = 0;
  while (true) {
    bool progress = false;
    tr.count(TR_P_ITER);
    const long long t_it = tr.now();
    if (!done && !have) {
      if ((int)(ld_acquire_cta(&e.ctrl->desc_hi) - p) > 0) {
        const PhaseDesc* d = desc_slot(e, p);
        kf = d->kind_flags;
        progress = true;
        if ((kf & 15u) == DK_END) done = true;
        else {
          KT = d->KT; T = d->T; kt0 = d->kt0; N = d->S * T;
          item_range<CW>(N, w, i0, i1);
          if (i0 == i1) ++p;
          else {
            have = true;
            const uint32_t fmt = (kf >> 4) & 3u;
            rec_bytes = fmt == FMT_SQ3 ? (uint32_t)RWKVQ_SQ_RECORD_BYTES : fmt == FMT_VQ6 ? 1536u : 2048u;
            cb_bytes = fmt == FMT_SQ3 ? 0u : fmt == FMT_VQ6 ? 256u : 1024u;
            xoff = a.off_x + d->xoff; gsoff = a.off_x + d->gsoff; row0 = d->row0;
            cnt_base = d->cnt_base; src0 = d->src; cb0 = d->cb;
            sl0 = i0 / T;
            i = i0;
          }
        }
      }
    } else if (!done) {
      if (n - tail >= (uint32_t)kHeaderRing) tail = ld_acquire_cta(&e.ctrl->hq_tail[w]);
      if (n - tail < (uint32_t)kHeaderRing) {
        progress = true;
        const uint32_t sl = i / T, tt = i - sl * T;
        const uint32_t lo = sl * T, hi = lo + T;
        const uint32_t iend = min(i1, hi);                 // the run: items [i, iend) of slice sl
        const uint32_t kt = kt0 + tt;
        const uint32_t row = row0 + 16u * sl;
        const uint64_t src = src0 + (uint64_t)((row >> 7) * KT + kt) * (8u * rec_bytes) + ((row >> 4) & 7u) * rec_bytes;
        const uint64_t cbs = cb0 + (uint64_t)((row >> 8) * KT + kt) * cb_bytes;
        // who else holds a part of the slice
        uint32_t wlo, whi;
        if (N >= (uint32_t)CW) { wlo = ((lo + 1u) * (uint32_t)CW + N - 1u) / N - 1u; whi = (hi * (uint32_t)CW + N - 1u) / N - 1u; }
        else { wlo = lo; whi = hi - 1u; }
        uint32_t f0, f1;
        item_range<CW>(N, wlo, f0, f1);
        uint32_t flags = (iend - i) | (((cnt_base + sl) & (uint32_t)(kCnt - 1)) << 9) | ((whi - wlo + 1u) << 16) | (wlo << 24);
        if (sl != sl0) flags |= IF_RSELF;
        if (f0 < lo) flags |= IF_RFIRST;
        uint4* h = reinterpret_cast<uint4*>(hq + (size_t)(n % (uint32_t)kHeaderRing) * 32u);
        h[0] = make_uint4(xoff + tt * 512u, gsoff + tt * sums_tile, flags, row);
        h[1] = make_uint4((uint32_t)src | ((kf >> 4) & 3u), (uint32_t)(src >> 32), (uint32_t)(cbs - src), 0u);
        ++n;
        st_release_cta(&e.ctrl->hq_head[w], n);
        tr.count(TR_P_ISSUED);
        i = iend;
        if (i == i1) { have = false; ++p; }
      }
    }
    {
      // the oldest descriptor any lane still reads (lanes that are done, or unused, do not hold one back)
      const uint32_t pmin = __reduce_min_sync(0xFFFFFFFFu, done ? 0xFFFFFFFFu : p);
      if (pmin != last_pmin && pmin != 0xFFFFFFFFu) { last_pmin = pmin; if (w == 0) st_release_cta(&e.ctrl->prod_tail, pmin); }
    }
    if (__all_sync(0xFFFFFFFFu, done)) break;
    if (__any_sync(0xFFFFFFFFu, progress)) { idle = 0; tr.add(TR_P_WORK, t_it); continue; }
    tr.count(TR_P_IDLE);
    if (*e.abortp) break;
    if (++idle > (a.poll_limit << 4)) { give_up(e); break; }
    __nanosleep(100);
  }
  tr.add(TR_P_TOTAL, t_begin);
  tr.store(a.trace);
}


// ---- the flag barrier -----------------------------------------------------------------------------

// All of this warp's lanes together read every CTA's word; true once all have reached `target`.
__device__ __forceinline__ bool flags_reached(const unsigned* flags, int P, unsigned target, int lane) {
  // Acquire loads (an acquire load costs about what a relaxed one does, a separate fence after the
  // poll three times as much); every load is issued before the first result is looked at: one
  // round trip per poll.
  unsigned behind = 0u;
  for (int c = lane; c < P; c += 32) behind |= (ld_acquire_gpu(flags + c) - target) >> 31;
  return __all_sync(0xFFFFFFFFu, behind == 0u);
}
__device__ __forceinline__ bool flags_wait(const Env& e, const unsigned* flags, unsigned target, int lane) {
  const int P = (int)gridDim.x;
  for (uint32_t it = 0; it < (e.a.poll_limit << 2); ++it) {
    if (flags_reached(flags, P, target, lane)) return true;
    if ((it & 7u) == 7u && *e.abortp) return false;
  }
  if (lane == 0) give_up(e);
  return false;
}

// ---- auxiliary warp: descriptor ring, barrier detection -------------------------------------------
template <bool TRACE>
__device__ void aux_role(const Env& e) {
  const StepArgs& a = e.a;
  const int lane = threadIdx.x & 31;
  Tracer<TRACE> tr;
  const long long t_begin = tr.now();
  const uint32_t d0 = a.desc_off[blockIdx.x], n_desc = a.desc_off[blockIdx.x + 1] - d0;
  uint32_t hi = 0;
  auto refill = [&]() {
    // copy descriptors into the ring as far as the other warps' progress allows, four per pass
    const uint32_t tail = min(ld_acquire_cta(&e.ctrl->desc_tail), ld_acquire_cta(&e.ctrl->prod_tail));
    bool any = false;
    while (hi < n_desc && hi < tail + (uint32_t)kDescRing) {
      const uint32_t k = hi + (uint32_t)(lane >> 3);
      if (k < n_desc && k < tail + (uint32_t)kDescRing) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(a.descs + d0 + k) + (lane & 7));
        *(reinterpret_cast<uint4*>(const_cast<PhaseDesc*>(desc_slot(e, k))) + (lane & 7)) = v;
      }
      hi = min(min(hi + 4u, n_desc), tail + (uint32_t)kDescRing);
      any = true;
    }
    if (any) {
      __syncwarp();
      if (lane == 0) st_release_cta(&e.ctrl->desc_hi, hi);
    }
  };
  if (lane == 0 && a.init_post[blockIdx.x]) st_relaxed_gpu(a.flags + blockIdx.x, a.base + a.init_post[blockIdx.x]);
  refill();
  for (uint32_t p = 0; p < n_desc; ++p) {
    if (p >= hi) {
      // the ring is full of descriptors the other warps still need: wait for them to move on
      bool ok = false;
      for (uint32_t it = 0; it < (a.poll_limit << 4); ++it) {
        refill();
        if (p < hi) { ok = true; break; }
        if ((it & 63u) == 63u && *e.abortp) break;
        __nanosleep(100);
      }
      if (!ok) { if (lane == 0 && !*e.abortp) give_up(e); return; }
    }
    const PhaseDesc* d = desc_slot(e, p);
    const uint32_t kf = d->kind_flags;
    if ((kf & 15u) == DK_END) break;
    if (kf & DF_FIRST) {
      // the stage may start once every CTA has completed all earlier stages
      const uint32_t stage = d->stage;
      const long long t0 = tr.now();
      if (stage > 0u && !flags_wait(e, a.flags, a.base + stage + a.wait_skew, lane)) return;
      tr.add(TR_A_WAIT, t0); tr.count(TR_A_POLLS);
      if (lane == 0) Tracer<TRACE>::stamp(a.trace, stage, 1);
      __syncwarp();
      if (lane == 0) mbar_arrive(&e.ctrl->open);
    }
    {
      const long long t0 = tr.now();
      refill();
      tr.add(TR_A_REFILL, t0);
    }
  }
  tr.add(TR_A_TOTAL, t_begin);
  tr.store(a.trace);
}

// ---- consumer warps: input staging ------------------------------------------------------------------

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
// mu_hat of the eight columns col..col+7 (col a multiple of 8): four 2-D codebook entries whose
// indices start at a byte boundary of the index stream.
__device__ __forceinline__ uint4 mu_vector(const uint8_t* mu, const uint8_t* mu_aux, uint32_t bits, int col) {
  const uint32_t mask = (1u << bits) - 1u;
  const uint32_t byte = (uint32_t)(col >> 1) * bits >> 3;
  const uint32_t* w = reinterpret_cast<const uint32_t*>(mu) + (byte >> 2);
  const uint32_t sh = (byte & 3u) * 8u;
  const uint32_t lo = __ldg(w);
  const uint32_t hi = (sh + 4u * bits > 32u) ? __ldg(w + 1) : 0u;
  const uint32_t f = __funnelshift_r(lo, hi, sh);
  const uint32_t* cb = reinterpret_cast<const uint32_t*>(mu_aux);
  return make_uint4(__ldg(cb + (f & mask)), __ldg(cb + ((f >> bits) & mask)), __ldg(cb + ((f >> (2 * bits)) & mask)),
                    __ldg(cb + ((f >> (3 * bits)) & mask)));
}
// The three sums of a 128-column group the factored dequantisation needs, from the rounded fp16
// values the tensor core will see: Sx = sum x and, negated, Bx_h = sum bias_h(col) * x for the two
// row halves of a record.  Called by a half-warp whose lane l16 holds columns 8*l16..8*l16+7.
__device__ __forceinline__ void group_sums(const uint4 v, int l16, float& sx, float& nb0, float& nb1) {
  const int o = (8 * l16) & 63;
  const float pa = pair_sum(v.x) + pair_sum(v.z), pb = pair_sum(v.y) + pair_sum(v.w);
  sx = pa + pb;
  nb0 = -fmaf((float)rwkvq_sq_bias(o, 0), pa, (float)rwkvq_sq_bias(o + 2, 0) * pb);
  nb1 = -fmaf((float)rwkvq_sq_bias(o, 1), pa, (float)rwkvq_sq_bias(o + 2, 1) * pb);
#pragma unroll
  for (int d = 8; d > 0; d >>= 1) {
    sx += __shfl_xor_sync(0xFFFFFFFFu, sx, d);
    nb0 += __shfl_xor_sync(0xFFFFFFFFu, nb0, d);
    nb1 += __shfl_xor_sync(0xFFFFFFFFu, nb1, d);
  }
}

// The consumer threads of a CTA mix the inputs of the phases [p0, p1) of a staging group into the
// input area.  A thread owns 16-byte vectors (8 columns of one batch row of a slab) tid, tid + NT,
// ... of the concatenated phases; x_prev and mu_hat of its first two vectors can be fetched BEFORE
// the grid barrier is awaited, so that only one round of loads of x, the mix and the sums follow it.
template <int CW>
struct Stager {
  static constexpr int NT = CW * 32, PRE = 2;
  uint4 xp[PRE], mh[PRE];

  // vector number v of the group -> phase, batch row, vector within the slab's row
  __device__ __forceinline__ static const PhaseDesc* locate(const Env& e, uint32_t p0, uint32_t p1, int B, uint32_t v, int& b, int& c8) {
    for (uint32_t p = p0; p < p1; ++p) {
      const PhaseDesc* d = desc_slot(e, p);
      const uint32_t nvr = d->T * 32u, nv = (uint32_t)B * nvr;
      if (v < nv) { b = (int)(v / nvr); c8 = (int)(v - (uint32_t)b * nvr); return d; }
      v -= nv;
    }
    return nullptr;
  }
  __device__ __forceinline__ void before_barrier(const Env& e, uint32_t p0, uint32_t p1) {
#pragma unroll
    for (int k = 0; k < PRE; ++k) {
      int b, c8;
      const PhaseDesc* d = locate(e, p0, p1, e.a.B, (uint32_t)(threadIdx.x + k * NT), b, c8);
      xp[k] = make_uint4(0u, 0u, 0u, 0u); mh[k] = xp[k];
      if (d && (d->kind_flags & DF_MU)) {
        const int col = (int)d->kt0 * 256 + 8 * c8;
        if (col < (int)d->ic) {
          xp[k] = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(d->xprev) + (size_t)b * d->ic + col));
          mh[k] = mu_vector(reinterpret_cast<const uint8_t*>(d->mu), reinterpret_cast<const uint8_t*>(d->mu_aux), d->mu_bits, col);
        }
      }
    }
  }
  // Mix, round and store one vector; reduce the group's sums.  Called by whole warps.
  __device__ __forceinline__ static void finish_vector(const Env& e, const PhaseDesc* d, int b, int c8, bool pre, uint4 pr, uint4 m) {
    const int lane = threadIdx.x & 31, nbp = e.a.nbp;
    uint8_t* xarea = e.smem + e.a.off_x;
    const int col = (int)d->kt0 * 256 + 8 * c8;
    uint4 r = make_uint4(0u, 0u, 0u, 0u);
    if (col < (int)d->ic) {
      r = __ldcg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(d->x) + (size_t)b * d->ic + col));
      if (d->kind_flags & DF_MU) {
        if (!pre) {
          pr = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(d->xprev) + (size_t)b * d->ic + col));
          m = mu_vector(reinterpret_cast<const uint8_t*>(d->mu), reinterpret_cast<const uint8_t*>(d->mu_aux), d->mu_bits, col);
        }
        r.x = mix2(r.x, pr.x, m.x); r.y = mix2(r.y, pr.y, m.y); r.z = mix2(r.z, pr.z, m.z); r.w = mix2(r.w, pr.w, m.w);
      }
    }
    *reinterpret_cast<uint4*>(xarea + d->xoff + (size_t)b * d->xstride + (size_t)c8 * 16) = r;
    if (d->kind_flags & DF_SUMS) {
      float sx, nb0, nb1;
      group_sums(r, lane & 15, sx, nb0, nb1);
      if ((lane & 15) == 0) {
        float* gs = reinterpret_cast<float*>(xarea + d->gsoff);
        const int grp = c8 >> 4;
        gs[(grp * 3 + 0) * nbp + b] = sx;
        gs[(grp * 3 + 1) * nbp + b] = nb0;
        gs[(grp * 3 + 2) * nbp + b] = nb1;
      }
    }
  }
  // A row is a multiple of 32 vectors, so a warp is inside one row of one phase or past the end:
  // every branch below is warp-uniform.  `pre`: before_barrier has run for this group.
  __device__ __forceinline__ void stage(const Env& e, uint32_t p0, uint32_t p1, bool pre) {
#pragma unroll
    for (int k = 0; k < PRE; ++k) {
      int b = 0, c8 = 0;
      const PhaseDesc* d = locate(e, p0, p1, e.a.B, (uint32_t)(threadIdx.x + k * NT), b, c8);
      if (!d) return;
      finish_vector(e, d, b, c8, pre, xp[k], mh[k]);
    }
    for (int k = PRE;; ++k) {
      int b = 0, c8 = 0;
      const PhaseDesc* d = locate(e, p0, p1, e.a.B, (uint32_t)(threadIdx.x + k * NT), b, c8);
      if (!d) return;
      finish_vector(e, d, b, c8, false, make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u));
    }
  }
};

// ---- consumer warps: the record loop ------------------------------------------------------------------

// One 128-column group of an SQ record (16 rows) against the staged input:
//   acc[b][row] += s * ( sum_cols (q+bias) x  -  Bx_h  -  z * Sx )
// Two chains of four m16n8k16 steps each (even and odd steps) keep the dependent tensor-core
// latency short; the first starts at -Bx_h (the bias every extracted half carries, from the
// precomputed sums), so that after the steps only an add and two FMAs per output remain.
// `w`: the group's six words; sz_lo / sz_hi: (s, z) fp16 pairs of rows g and g+8; xa[n]: byte
// offset in shared memory of this lane's fragment of batch block n at the group's first column;
// gs: byte offset of this lane's part of the group's sums [3][nbp].
template <int NB>
__device__ __forceinline__ void sq_group(const uint32_t (&w)[6], uint32_t sz_lo, uint32_t sz_hi, const uint32_t (&xa)[NB],
                                         uint32_t gs, uint32_t gstride, float (&acc)[NB][4]) {
  float c0[NB][4], c1[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const float2 b0 = *reinterpret_cast<const float2*>(smem_base + gs + gstride + n * 32);
    const float2 b1 = *reinterpret_cast<const float2*>(smem_base + gs + 2 * gstride + n * 32);
    c0[n][0] = b0.x; c0[n][1] = b0.y; c0[n][2] = b1.x; c0[n][3] = b1.y;
    c1[n][0] = c1[n][1] = c1[n][2] = c1[n][3] = 0.f;
  }
#pragma unroll
  for (int ti = 0; ti < 2; ++ti) {
    uint32_t r[16];
    sq_unpack_triple(w[3 * ti], w[3 * ti + 1], w[3 * ti + 2], r);
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const uint32_t afrag[4] = {r[4 * m], r[4 * m + 1], r[4 * m + 2], r[4 * m + 3]};
#pragma unroll
      for (int n = 0; n < NB; ++n) {
        const uint2 bf = *reinterpret_cast<const uint2*>(smem_base + xa[n] + (4 * ti + m) * 32);
        if (m & 1) mma_16816(c1[n], afrag, bf.x, bf.y); else mma_16816(c0[n], afrag, bf.x, bf.y);
      }
    }
  }
  const uint32_t nlo = sz_lo ^ 0x80000000u, nhi = sz_hi ^ 0x80000000u;   // (s, -z)
  const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&nlo));
  const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&nhi));
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const float2 sx = *reinterpret_cast<const float2*>(smem_base + gs + n * 32);
    acc[n][0] = fmaf(s0.x, fmaf(s0.y, sx.x, c0[n][0] + c1[n][0]), acc[n][0]);
    acc[n][1] = fmaf(s0.x, fmaf(s0.y, sx.y, c0[n][1] + c1[n][1]), acc[n][1]);
    acc[n][2] = fmaf(s1.x, fmaf(s1.y, sx.x, c0[n][2] + c1[n][2]), acc[n][2]);
    acc[n][3] = fmaf(s1.x, fmaf(s1.y, sx.y, c0[n][3] + c1[n][3]), acc[n][3]);
  }
}

// Eight tensor-core steps (HALF of a tile's columns) of a VQ record: every fragment register is one
// lookup in the tile's codebook, which sits behind the record in the ring entry.
template <int BITS, int NB, int HALF>
__device__ __forceinline__ void vq_half(const uint32_t (&w)[2 * BITS], const uint32_t* cb, const uint32_t (&xa)[NB],
                                        float (&acc)[NB][4]) {
#pragma unroll
  for (int j = 8 * HALF; j < 8 * HALF + 8; ++j) {
    uint32_t afrag[4];
#pragma unroll
    for (int R = 0; R < 4; ++R) afrag[R] = cb[vq_index<BITS, 2 * BITS>(w, 4 * j + R)];
#pragma unroll
    for (int n = 0; n < NB; ++n) {
      const uint2 bf = *reinterpret_cast<const uint2*>(smem_base + xa[n] + j * 32);
      mma_16816(acc[n], afrag, bf.x, bf.y);
    }
  }
}

// 16-byte asynchronous copies global -> shared in per-thread groups.
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src, uint64_t policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "l"(policy) : "memory");
}
// The same copy by the lanes for which `on` holds, as one predicated instruction (no divergent branch).
__device__ __forceinline__ void cp_async16_if(bool on, uint32_t dst_smem, const void* src, uint64_t policy) {
  asm volatile("{\n .reg .pred p;\n setp.ne.u32 p, %3, 0;\n @p cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n}"
               ::"r"(dst_smem), "l"(src), "l"(policy), "r"((uint32_t)on) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// Wait until at most `pending` (0..6) of this thread's most recent groups are still in flight.
__device__ __forceinline__ void cp_async_wait_pending(uint32_t pending) {
  switch (pending) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
    case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
  }
}

// What a consumer warp carries from record to record.
template <int NB>
struct ConsumerState {
  float acc[NB][4];
  uint32_t infl;               // records whose copies are issued and not yet consumed
  uint32_t slot, islot;        // ring entry of the next record to consume / to issue
  uint32_t run_cons, run_iss;  // run headers read by the consuming / by the issuing side
  const uint8_t* iss_src;      // issuing side: this lane's part of the next record of the current run
  uint32_t iss_cb;             // ... its codebook, as an offset from iss_src (VQ)
  uint32_t iss_left, iss_fmt;  // ... records left in the run; the run's format
  int rowsel[NB];
};

template <int NB, int CW, bool TRACE>
struct Consumer {
  const Env& e;
  Tracer<TRACE>& tr;
  ConsumerState<NB>& s;
  const uint32_t w, lane, g, t, depth, entry, ring, hq;   // ring / hq: byte offsets in shared memory
  const uint64_t policy;

  // Issue the copies of the next record (and of the codebook behind it) into ring entry islot as one
  // group.  The entry is free: the warp itself has consumed what was in it.  When the current run is
  // exhausted the next run header is taken, if the producer lane has written it.
  __device__ __forceinline__ bool issue_one() {
    if (s.iss_left == 0u) {
      if ((int)(ld_acquire_cta(&e.ctrl->hq_head[w]) - s.run_iss) <= 0) return false;
      const uint32_t hoff = hq + (s.run_iss % (uint32_t)kHeaderRing) * 32u;
      const uint4 q1 = *reinterpret_cast<const uint4*>(smem_base + hoff + 16u);
      s.iss_left = *reinterpret_cast<const uint32_t*>(smem_base + hoff + 8u) & 0x1FFu;
      s.iss_fmt = q1.x & 3u;
      s.iss_src = reinterpret_cast<const uint8_t*>(((uint64_t)q1.y << 32) | (q1.x & ~15u)) + lane * 16u;
      s.iss_cb = q1.z;
      ++s.run_iss;
    }
    const uint8_t* src = s.iss_src;
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_base) + ring + s.islot * entry + lane * 16u;
    cp_async16(dst, src, policy);
    cp_async16(dst + 512u, src + 512, policy);
    cp_async16(dst + 1024u, src + 1024, policy);
    if (s.iss_fmt == FMT_SQ3) {
      cp_async16_if(lane < 8u, dst + 1536u, src + 1536, policy);
      s.iss_src = src + 8 * RWKVQ_SQ_RECORD_BYTES;
    } else if (s.iss_fmt == FMT_VQ6) {
      cp_async16_if(lane < 16u, dst + 1536u, src + s.iss_cb, policy);
      s.iss_src = src + 8 * 1536; s.iss_cb += 256u - 8u * 1536u;
    } else {
      cp_async16(dst + 1536u, src + 1536, policy);
      cp_async16(dst + 2048u, src + s.iss_cb, policy);
      cp_async16(dst + 2560u, src + s.iss_cb + 512, policy);
      s.iss_src = src + 8 * 2048; s.iss_cb += 1024u - 8u * 2048u;
    }
    cp_async_commit();
    --s.iss_left; ++s.infl;
    if (++s.islot == depth) s.islot = 0;
    return true;
  }
  __device__ __forceinline__ void top_up() { while (s.infl < depth && issue_one()) {} }

  // The rows of a finished slice: vals[j] holds element lane + 32*j of the slice's [batch][16 rows]
  // block, summed over this CTA's slab.  One slab: these are the outputs.  Several: the sums go to
  // the slab's scratch slot, and the last slab to arrive adds all slabs in slab order and stores the
  // rows.
  __device__ __forceinline__ void finish_slice(const PhaseDesc* d, uint32_t row, const float (&vals)[kMaxVals]) {
    const StepArgs& a = e.a;
    float* y = reinterpret_cast<float*>(d->y);
    const uint32_t oc = d->oc, ks = d->ks_part & 0xFFFFu, nel = 16u * (uint32_t)a.B;
    if (ks == 1u) {
#pragma unroll
      for (int j = 0; j < kMaxVals; ++j) {
        const uint32_t el = lane + 32u * j;
        if (el < nel) y[(size_t)(el >> 4) * oc + row + (el & 15u)] = vals[j];
      }
      return;
    }
    const uint32_t slot = d->gslot0 + ((row - d->row0) >> 4) * ks;
    float* mine = a.gpart + (size_t)(slot + (d->ks_part >> 16)) * a.slot_floats;
#pragma unroll
    for (int j = 0; j < kMaxVals; ++j) {
      const uint32_t el = lane + 32u * j;
      if (el < nel) __stcg(mine + el, vals[j]);
    }
    // every lane's stores precede lane 0's release; whoever finds all the other slabs arrived
    // acquires their stores with the same operation
    __syncwarp();
    unsigned old = 0;
    if (lane == 0) old = atom_add_acq_rel_gpu(a.gcnt + slot, 1u);
    old = __shfl_sync(0xFFFFFFFFu, old, 0);
    __syncwarp();
    if (old + 1u == ks) {
      if (lane == 0) a.gcnt[slot] = 0u;      // the next use lies behind a stage barrier
      const float* all = a.gpart + (size_t)slot * a.slot_floats;
#pragma unroll
      for (int j = 0; j < kMaxVals; ++j) {
        const uint32_t el = lane + 32u * j;
        if (el < nel) {
          float sum = 0.f;
          for (uint32_t k = 0; k < ks; ++k) sum += __ldcg(all + (size_t)k * a.slot_floats + el);
          y[(size_t)(el >> 4) * oc + row + (el & 15u)] = sum;
        }
      }
    }
  }

  // The warp's n_runs runs of one phase, all of format FMT.  False after a failed wait.
  template <int FMT>
  __device__ __forceinline__ bool run(const PhaseDesc* d, uint32_t n_runs) {
    const StepArgs& a = e.a;
    const uint32_t gstride = (uint32_t)a.nbp * 4u, sums_tile = 6u * gstride;
    const uint32_t slot0 = d->slot_set * 2u * (uint32_t)CW;
    float* partial = reinterpret_cast<float*>(smem_base + a.off_partial);
    uint32_t lane_x[NB];      // this lane's part of a fragment address: batch row and column quad
#pragma unroll
    for (int n = 0; n < NB; ++n) lane_x[n] = t * 8u + (uint32_t)s.rowsel[n] * d->xstride;
    for (uint32_t r = 0; r < n_runs; ++r) {
      // the run's header: the producer lane is normally far ahead; wait for it (bounded) if not
      if ((int)(ld_acquire_cta(&e.ctrl->hq_head[w]) - s.run_cons) <= 0) {
        bool ok = false;
        for (uint32_t k = 0; k < (a.poll_limit << 4); ++k) {
          if ((int)(ld_acquire_cta(&e.ctrl->hq_head[w]) - s.run_cons) > 0) { ok = true; break; }
          if ((k & 63u) == 63u && *e.abortp) break;
          __nanosleep(32);
        }
        if (!ok) { if (!*e.abortp) give_up(e); return false; }
      }
      const uint4 ha = *reinterpret_cast<const uint4*>(smem_base + hq + (s.run_cons % (uint32_t)kHeaderRing) * 32u);
      const uint32_t flags = ha.z, n_items = flags & 0x1FFu;
      uint32_t xa[NB];
#pragma unroll
      for (int n = 0; n < NB; ++n) xa[n] = ha.x + lane_x[n];
      uint32_t gs = ha.y + t * 8u;
#pragma unroll
      for (int n = 0; n < NB; ++n)
#pragma unroll
        for (int k = 0; k < 4; ++k) s.acc[n][k] = 0.f;
      for (uint32_t it = 0; it < n_items; ++it) {
        const long long t_w = tr.now();
        if (s.infl == 0u) issue_one();                  // its header is there: cannot fail
        cp_async_wait_pending(s.infl - 1u);
        __syncwarp();                                   // every lane's part of the record has landed
        tr.add(TR_WAIT_FULL, t_w);
        const long long t_i = tr.now();
        tr.count(TR_NITEMS);
        const uint32_t rec = ring + s.slot * entry;
        if (FMT == FMT_SQ3) {
          const uint4 p0 = *reinterpret_cast<const uint4*>(smem_base + rec + lane * 16u);
          const uint4 p1 = *reinterpret_cast<const uint4*>(smem_base + rec + 512u + lane * 16u);
          const uint4 p2 = *reinterpret_cast<const uint4*>(smem_base + rec + 1024u + lane * 16u);
          const uint4 sz = *reinterpret_cast<const uint4*>(smem_base + rec + (uint32_t)RWKVQ_SQ_CODE_BYTES + g * 16u);
          // the record is in registers: once every lane has read its part, the entry is refilled
          __syncwarp();
          --s.infl; if (++s.slot == depth) s.slot = 0;
          issue_one();
          {
            const uint32_t w0[6] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y};
            sq_group<NB>(w0, sz.x, sz.z, xa, gs, gstride, s.acc);
          }
          {
            uint32_t xb[NB];
#pragma unroll
            for (int n = 0; n < NB; ++n) xb[n] = xa[n] + 256u;
            const uint32_t w1[6] = {p1.z, p1.w, p2.x, p2.y, p2.z, p2.w};
            sq_group<NB>(w1, sz.y, sz.w, xb, gs + 3u * gstride, gstride, s.acc);
          }
        } else {
          const uint8_t* recp = smem_base + rec;
          if (FMT == FMT_VQ6) {
            const uint32_t* cb = reinterpret_cast<const uint32_t*>(recp + 1536);
            uint32_t v[12];
            vq_half_words<6, 0>(recp, (int)lane, v);
            vq_half_words<6, 1>(recp, (int)lane, v);
            vq_half<6, NB, 0>(v, cb, xa, s.acc);
            vq_half<6, NB, 1>(v, cb, xa, s.acc);
          } else {
            const uint32_t* cb = reinterpret_cast<const uint32_t*>(recp + 2048);
            uint32_t v[16];
            vq_half_words<8, 0>(recp, (int)lane, v);
            vq_half<8, NB, 0>(v, cb, xa, s.acc);
            vq_half_words<8, 1>(recp, (int)lane, v);
            vq_half<8, NB, 1>(v, cb, xa, s.acc);
          }
          // the codebook is looked up in the entry until the last step
          __syncwarp();
          --s.infl; if (++s.slot == depth) s.slot = 0;
          issue_one();
        }
#pragma unroll
        for (int n = 0; n < NB; ++n) xa[n] += 512u;
        gs += sums_tile;
        tr.add(TR_ITEMS, t_i);
      }
      // The header is no longer needed by either side (the issuing side is past it): tell the producer lane.
      ++s.run_cons;
      st_release_cta(&e.ctrl->hq_tail[w], s.run_cons);   // every lane stores the same word
      const long long t_f = tr.now();
      {
        // The run's sums leave the registers through a slot of shared memory in [batch][16 rows]
        // order: this warp's slot alone if the slice is its alone, else every holder's slot, added
        // in warp order by whoever writes last.
        const uint32_t ncon = (flags >> 16) & 0xFFu;
        float* ps = partial + (size_t)(slot0 + 2u * w + ((flags >> 29) & 1u)) * a.slot_floats;
#pragma unroll
        for (int n = 0; n < NB; ++n)
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int b = n * 8 + 2 * (int)t + (k & 1);
            if (b < a.B) ps[b * 16 + (int)g + 8 * (k >> 1)] = s.acc[n][k];
          }
        __syncwarp();
        bool last = true;
        uint32_t wlo = w, rfirst = (flags >> 29) & 1u;
        if (ncon > 1u) {
          uint32_t old = 0;
          uint32_t* cnt = &e.ctrl->cnt[(flags >> 9) & (uint32_t)(kCnt - 1)];
          if (lane == 0) old = smem_add_acq_rel(cnt, 1u);
          old = __shfl_sync(0xFFFFFFFFu, old, 0);
          __syncwarp();
          last = old + 1u == ncon;
          if (last && lane == 0) *cnt = 0u;
          wlo = (flags >> 24) & 31u; rfirst = (flags >> 30) & 1u;
        }
        if (last) {
          float vals[kMaxVals];
#pragma unroll
          for (int j = 0; j < kMaxVals; ++j) {
            const uint32_t el = lane + 32u * j;
            float sum = 0.f;
            if (el < 16u * (uint32_t)a.B)
              for (uint32_t k = 0; k < ncon; ++k)
                sum += partial[(size_t)(slot0 + 2u * (wlo + k) + (k == 0u ? rfirst : 0u)) * a.slot_floats + el];
            vals[j] = sum;
          }
          finish_slice(d, ha.w, vals);
        }
      }
      tr.add(TR_FLUSH, t_f);
    }
    return true;
  }
};


template <int NB, int CW, bool TRACE>
__device__ void consumer_role(const Env& e) {
  const StepArgs& a = e.a;
  Tracer<TRACE> tr;
  const long long t_begin = tr.now();
  const uint32_t lane = threadIdx.x & 31u, w = threadIdx.x >> 5;
  ConsumerState<NB> s;
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    s.rowsel[n] = min(8 * n + (int)(lane >> 2), a.B - 1);
#pragma unroll
    for (int k = 0; k < 4; ++k) s.acc[n][k] = 0.f;
  }
  s.infl = s.slot = s.islot = s.run_cons = s.run_iss = 0u;
  s.iss_src = nullptr; s.iss_cb = 0u; s.iss_left = 0u; s.iss_fmt = 0u;
  Consumer<NB, CW, TRACE> c{e, tr, s, w, lane, lane >> 2, lane & 3u, (uint32_t)a.depth, a.entry_bytes,
                            a.off_ring + w * (uint32_t)a.depth * a.entry_bytes, a.off_hq + w * (uint32_t)kHeaderRing * 32u,
                            policy_evict_first()};
  uint32_t opened = 0;                 // stages this CTA has taken part in
  uint32_t reported = 0;               // stages this warp has left
  bool dead = false, verdict = false;  // verdict: the role's barrier has already told everyone to leave
  Stager<CW> stager;

  for (uint32_t p = 0;; ++p) {
    {
      const long long t0 = tr.now();
      if (!wait_desc(e, p)) dead = true;
      tr.add(TR_WAIT_DESC, t0);
    }
    if (dead) break;
    const PhaseDesc* d = desc_slot(e, p);
    const uint32_t kf = d->kind_flags;
    if ((kf & 15u) == DK_END) break;
    c.top_up();                        // the weight ring, before anything that may wait
    if (kf & DF_GROUP) {
      uint32_t p1 = p + 1;
      while (true) {                   // the group's phases: p .. the one flagged last
        if (!wait_desc(e, p1 - 1)) { dead = true; break; }
        if (desc_slot(e, p1 - 1)->kind_flags & DF_GLAST) break;
        ++p1;
      }
      if (dead) break;
      if (kf & DF_FIRST) {
        {
          const long long t0 = tr.now();
          stager.before_barrier(e, p, p1);
          tr.add(TR_PRE, t0);
        }
        {
          const long long t0 = tr.now();
          if (!mbar_wait(e, &e.ctrl->open, opened & 1u)) dead = true;
          tr.add(TR_WAIT_OPEN, t0);
          if (threadIdx.x == 0) Tracer<TRACE>::stamp(a.trace, d->stage, 2);
        }
        ++opened;
      } else {
        // a later group of the stage reuses the input area: every warp must have left the earlier one
        if (!named_bar_and(1, CW * 32, true)) { dead = true; verdict = true; break; }
      }
      const long long t1 = tr.now();
      if (!dead) stager.stage(e, p, p1, (kf & DF_FIRST) != 0u);
      // every consumer thread's stores precede the verdict; all leave together after a failure
      if (!named_bar_and(1, CW * 32, !dead)) { dead = true; verdict = true; break; }
      tr.add(TR_POST, t1);
      if ((kf & DF_FIRST) && threadIdx.x == 0) {
        Tracer<TRACE>::stamp(a.trace, d->stage, 3);
        st_release_cta(&e.ctrl->desc_tail, p);
      }
    } else if (kf & DF_SYNC) {
      // the phase reuses partial-sum slots or slice counters of an earlier phase of this stage: every
      // warp must have left that phase (its slices are then reduced and stored)
      if (!named_bar_and(1, CW * 32, true)) { dead = true; verdict = true; break; }
    }
    uint32_t i0, i1;
    item_range<CW>(d->S * d->T, w, i0, i1);
    const uint32_t n_runs = i1 > i0 ? (i1 - 1u) / d->T - i0 / d->T + 1u : 0u;   // slices the warp's share touches
    const uint32_t fmt = (kf >> 4) & 3u;
    bool ok;
    if (fmt == FMT_SQ3) ok = c.template run<FMT_SQ3>(d, n_runs);
    else if (fmt == FMT_VQ6) ok = c.template run<FMT_VQ6>(d, n_runs);
    else ok = c.template run<FMT_VQ8>(d, n_runs);
    if (!ok) { dead = true; break; }
    if (kf & DF_LAST) {
      // This warp has left the stage.  The count is an acquire-release read-modify-write at CTA scope
      // and the publication a GPU-scope release by whoever reports last, so it is ordered after
      // everything every warp stored before reporting: block-level synchronisation followed by one
      // thread's release, the pattern of a cooperative grid barrier.
      __syncwarp();
      if (lane == 0) {
        const uint32_t old = smem_add_acq_rel(&e.ctrl->warps_done, 1u);
        if (old + 1u == (uint32_t)CW * (reported + 1u)) {
          fence_gpu();
          st_relaxed_gpu(a.flags + blockIdx.x, a.base + d->post_value);
          Tracer<TRACE>::stamp(a.trace, d->stage, 0);
        }
      }
      ++reported;
    }
  }
  // no copy of this warp may still be landing when the CTA's shared memory is given up
  cp_async_wait_all();
  if (dead && !verdict) named_bar_and(1, CW * 32, false);   // keep the role's barrier whole: the others leave through this verdict
  tr.add(TR_TOTAL, t_begin);
  tr.store(a.trace);
}

template <int NB, int CW, bool TRACE>
__global__ void __launch_bounds__((CW + 2) * 32, 1) step_kernel(const StepArgs a) {
  uint8_t* smem = smem_base;
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem);
  if (threadIdx.x == 0) {
    mbar_init(&ctrl->open, 1);
    for (int k = 0; k < kMaxCW; ++k) { ctrl->hq_head[k] = 0u; ctrl->hq_tail[k] = 0u; }
    ctrl->warps_done = 0u; ctrl->desc_hi = 0u; ctrl->desc_tail = 0u; ctrl->prod_tail = 0u; ctrl->abort_flag = 0;
    for (int k = 0; k < kCnt; ++k) ctrl->cnt[k] = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const Env e{a, smem, ctrl, &ctrl->abort_flag};
  const int warp = threadIdx.x >> 5;
  if (warp < CW) consumer_role<NB, CW, TRACE>(e);
  else if (warp == CW) producer_role<CW, TRACE>(e);
  else aux_role<TRACE>(e);
}

// ---- host planner --------------------------------------------------------------------------------

struct PlanInfo {
  int P, B, NB, CW, depth, n_stages;
  unsigned runs;        // launches since the flags were last zero
  unsigned abort_epoch; // value of the abort epoch when the flags were last known good
  uint32_t poll_limit, wait_skew, n_sets;
  void* trace_dev;      // rwkvq_step_trace: where the next runs write their per-warp counters
  uint32_t entry_bytes, slot_floats, smem_bytes, off_hq, off_partial, off_x, off_ring;
  size_t off_desc_off, off_init_post, off_descs, off_flags, off_gcnt, off_gpart, total_bytes;
  uint32_t n_descs, gslots;
};

static std::mutex g_plan_mutex;
static std::unordered_map<const void*, PlanInfo> g_plans;

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
    if (o.y_dtype != RWKVQ_F32) return RWKVQ_EUNSUPPORTED;   // the step writes fp32 outputs
    if (i > 0 && o.stage < ops[i - 1].stage) return RWKVQ_EINVAL;
  }
  return RWKVQ_OK;
}

static int fmt_of(const rwkvq_desc& d) { return d.method == RWKVQ_SQ ? FMT_SQ3 : d.bits == 6 ? FMT_VQ6 : FMT_VQ8; }

// Input-area footprint of a slab of `cols` columns: B rows of fp16 values plus 32 bytes of padding
// each (the 8-byte fragment loads of a half-warp then hit 16 distinct bank pairs), the group
// sums, and 64 bytes of slack that lanes of batch columns which do not exist read (and discard).
static uint32_t xrows_bytes(int B, uint32_t cols) { return (uint32_t)B * (cols * 2u + 32u); }
static uint32_t xsums_bytes(int nbp, uint32_t cols, bool sums) { return sums ? (cols / 128u) * 3u * (uint32_t)nbp * 4u + 64u : 0u; }
static uint32_t xseg_bytes(int B, int nbp, uint32_t cols, bool sums) { return (xrows_bytes(B, cols) + xsums_bytes(nbp, cols, sums) + 15u) & ~15u; }

struct CtaPhase {
  int op;
  uint32_t slab, row0, S;
};

// Builds the whole plan on the host.  Returns the serialized image in `out` and fills `info`.
static rwkvq_status build_plan(const rwkvq_gemv_op* ops, int n_ops, int B, int P, std::vector<uint8_t>* out, PlanInfo* info) {
  rwkvq_status st = validate_ops(ops, n_ops, B);
  if (st != RWKVQ_OK) return st;
  const int NB = B <= 8 ? 1 : 2;
  const int CW = kConsumerWarps;
  const uint32_t nbp = (uint32_t)((B + 1) & ~1);
  info->P = P; info->B = B; info->NB = NB; info->CW = CW;
  info->poll_limit = kDefaultPollLimit; info->wait_skew = 0; info->trace_dev = nullptr;

  std::vector<std::pair<int, int>> stage_ranges;  // [first op, last op) per distinct stage value
  for (int i = 0; i < n_ops;) {
    int j = i;
    while (j < n_ops && ops[j].stage == ops[i].stage) ++j;
    stage_ranges.push_back({i, j});
    i = j;
  }
  const int n_stages = (int)stage_ranges.size();
  if (n_stages >= 65535) return RWKVQ_EUNSUPPORTED;
  info->n_stages = n_stages;

  // 1. K slabs: T tiles per slab, the largest divisor of KT whose inputs fit one segment of the input area
  const uint32_t kSegCap = 36u * 1024u, kAreaCap = B <= 8 ? 72u * 1024u : 36u * 1024u;
  std::vector<uint32_t> slab_tiles(n_ops, 1);
  for (int i = 0; i < n_ops; ++i) {
    const rwkvq_desc& d = ops[i].W_desc;
    const uint32_t KT = (uint32_t)d.ic_pad / 256u;
    for (uint32_t T = 1; T <= KT; ++T)
      if (KT % T == 0 && xseg_bytes(B, (int)nbp, T * 256u, d.method == RWKVQ_SQ) <= kSegCap) slab_tiles[i] = T;
  }

  // 2. deal every stage's (slab, 16-row slice) units to the CTAs: contiguous in (product, slab, row)
  //    order, balanced by cost (records x a weight per format: what a record costs a consumer warp)
  std::vector<std::vector<std::vector<CtaPhase>>> deal(n_stages, std::vector<std::vector<CtaPhase>>(P));
  for (int s = 0; s < n_stages; ++s) {
    uint64_t total = 0;
    auto unit_cost = [&](int o) -> uint64_t {
      const rwkvq_desc& d = ops[o].W_desc;
      const uint64_t wgt = d.method == RWKVQ_SQ ? 20u : d.bits == 8 ? 40u : 36u;
      return (uint64_t)slab_tiles[o] * wgt;
    };
    for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o)
      total += unit_cost(o) * (uint64_t)(ops[o].W_desc.oc / 16) * (uint64_t)((uint32_t)ops[o].W_desc.ic_pad / 256u / slab_tiles[o]);
    uint64_t run = 0;
    const int rot = (int)(((uint64_t)s * 37u) % (uint64_t)P);   // idle CTAs of small stages are not always the same SMs
    for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) {
      const uint64_t c1 = unit_cost(o);
      const int ns = ops[o].W_desc.oc / 16;
      const uint32_t ks = (uint32_t)ops[o].W_desc.ic_pad / 256u / slab_tiles[o];
      for (uint32_t k = 0; k < ks; ++k)
        for (int sl = 0; sl < ns; ++sl) {
          int c = (int)(((run + c1 / 2) * (uint64_t)P) / (total ? total : 1));
          if (c >= P) c = P - 1;
          c = (c + rot) % P;
          std::vector<CtaPhase>& L = deal[s][c];
          if (!L.empty() && L.back().op == o && L.back().slab == k && L.back().row0 + 16u * L.back().S == (uint32_t)sl * 16u) ++L.back().S;
          else L.push_back(CtaPhase{o, k, (uint32_t)sl * 16u, 1u});
          run += c1;
        }
    }
  }

  // 3. scratch slots of the products with several slabs (one region, reused by every stage: a slice's
  //    slots are read by the last slab to arrive before that CTA reports the stage)
  std::vector<uint32_t> gslot_base(n_ops, 0);
  uint32_t gslots = 0;
  for (int s = 0; s < n_stages; ++s) {
    uint32_t run = 0;
    for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) {
      const uint32_t ks = (uint32_t)ops[o].W_desc.ic_pad / 256u / slab_tiles[o];
      gslot_base[o] = run;
      if (ks > 1) run += (uint32_t)(ops[o].W_desc.oc / 16) * ks;
    }
    gslots = std::max(gslots, run);
  }
  info->gslots = gslots;

  // 4. per-CTA descriptor lists; the input area is as large as the largest staging group
  info->n_sets = B <= 3 ? 2u : 1u;
  uint32_t xarea = 0;
  std::vector<uint32_t> desc_off(P + 1, 0), init_post(P, 0);
  std::vector<PhaseDesc> descs;
  for (int c = 0; c < P; ++c) {
    desc_off[c] = (uint32_t)descs.size();
    // stages this CTA completes without consuming anything are reported with the previous stage
    // that has items (or at the start of the launch)
    std::vector<int> has_items(n_stages, 0);
    for (int s = 0; s < n_stages; ++s) has_items[s] = deal[s][c].empty() ? 0 : 1;
    int first_with = 0;
    while (first_with < n_stages && !has_items[first_with]) ++first_with;
    init_post[c] = (uint32_t)first_with;
    for (int s = 0; s < n_stages; ++s) {
      if (!has_items[s]) continue;
      std::vector<CtaPhase> phases;
      for (const CtaPhase& ph : deal[s][c])      // a phase's slices each own a counter
        for (uint32_t s0 = 0; s0 < ph.S; s0 += (uint32_t)kCnt)
          phases.push_back(CtaPhase{ph.op, ph.slab, ph.row0 + 16u * s0, std::min<uint32_t>((uint32_t)kCnt, ph.S - s0)});
      int next_with = s + 1;
      while (next_with < n_stages && !has_items[next_with]) ++next_with;
      uint32_t xo = 0, cnt = 0;
      for (size_t k = 0; k < phases.size(); ++k) {
        const CtaPhase& ph = phases[k];
        const rwkvq_gemv_op& op = ops[ph.op];
        const rwkvq_desc& d = op.W_desc;
        const uint8_t* img = static_cast<const uint8_t*>(op.W_image_dev);
        const bool sq = d.method == RWKVQ_SQ;
        const uint32_t T = slab_tiles[ph.op], KT = (uint32_t)d.ic_pad / 256u, ks = KT / T;
        const uint32_t seg = xseg_bytes(B, (int)nbp, T * 256u, sq);
        PhaseDesc pd;
        std::memset(&pd, 0, sizeof(pd));
        // the slice counters are reused once the stage has gone through all of them, the slots of
        // partial sums when the stage has more phases than sets: every warp must then have left the
        // phases that used them
        bool sync = k >= info->n_sets;
        if (cnt + ph.S > (uint32_t)kCnt) { cnt = 0; sync = true; }
        bool group = k == 0;
        if (xo + seg > kAreaCap) { group = true; xo = 0; }
        if (group && k > 0) descs.back().kind_flags |= DF_GLAST;
        pd.kind_flags = DK_PHASE | ((uint32_t)fmt_of(d) << 4) | (k == 0 ? DF_FIRST : 0u) | (k + 1 == phases.size() ? DF_LAST | DF_GLAST : 0u) |
                        (op.mu_image_dev ? DF_MU : 0u) | (sq ? DF_SUMS : 0u) | (sync ? DF_SYNC : 0u) | (group ? DF_GROUP : 0u);
        pd.slot_set = (uint32_t)(k % info->n_sets);
        pd.stage = (uint32_t)s;
        pd.src = (uint64_t)(uintptr_t)(img + RWKVQ_HEADER_BYTES);
        pd.cb = sq ? 0 : (uint64_t)(uintptr_t)(img + matrix_aux_offset(&d));
        pd.y = (uint64_t)(uintptr_t)op.y_dev;
        pd.oc = (uint32_t)d.oc; pd.row0 = ph.row0; pd.S = ph.S; pd.KT = KT;
        pd.T = T; pd.kt0 = ph.slab * T;
        pd.cnt_base = cnt; cnt += ph.S;
        pd.ks_part = ks | (ph.slab << 16);
        pd.gslot0 = gslot_base[ph.op] + (ph.row0 / 16u) * ks;
        pd.post_value = (uint32_t)next_with;
        pd.ic = (uint32_t)d.ic;
        pd.xoff = xo; pd.xstride = T * 512u + 32u;
        pd.gsoff = xo + xrows_bytes(B, T * 256u);
        xo += seg;
        xarea = std::max(xarea, xo);
        pd.x = (uint64_t)(uintptr_t)op.x_fp16_dev;
        if (op.mu_image_dev) {
          const uint8_t* mi = static_cast<const uint8_t*>(op.mu_image_dev);
          pd.xprev = (uint64_t)(uintptr_t)op.xprev_fp16_dev;
          pd.mu = (uint64_t)(uintptr_t)(mi + RWKVQ_HEADER_BYTES);
          pd.mu_aux = (uint64_t)(uintptr_t)(mi + vector_aux_offset(&op.mu_desc));
          pd.mu_bits = (uint16_t)op.mu_desc.bits; pd.mu_entries = (uint16_t)op.mu_desc.entries;
        }
        descs.push_back(pd);
      }
    }
    PhaseDesc end;
    std::memset(&end, 0, sizeof(end));
    end.kind_flags = DK_END;
    descs.push_back(end);
  }
  desc_off[P] = (uint32_t)descs.size();
  info->n_descs = (uint32_t)descs.size();

  // 5. shared-memory budget
  bool has_vq6 = false, has_vq8 = false;
  for (int i = 0; i < n_ops; ++i) {
    if (ops[i].W_desc.method == RWKVQ_SQ) continue;
    if (ops[i].W_desc.bits == 6) has_vq6 = true; else has_vq8 = true;
  }
  uint32_t entry = RWKVQ_SQ_RECORD_BYTES;
  if (has_vq6) entry = std::max(entry, 1536u + 256u);
  if (has_vq8) entry = std::max(entry, 2048u + 1024u);
  info->entry_bytes = entry;
  info->slot_floats = 16u * (uint32_t)B;
  info->off_hq = kCtrlBytes + kDescBytes;
  info->off_partial = info->off_hq + (uint32_t)CW * kHeaderRing * 32u;
  // Two sets of partial-sum slots where they are small, so that a CTA's second phase of a stage
  // starts without waiting for the first one's slices to be reduced.
  info->off_x = (info->off_partial + info->n_sets * 2u * (uint32_t)CW * info->slot_floats * 4u + 127u) & ~127u;
  xarea = (xarea + 127u) & ~127u;
  info->off_ring = info->off_x + xarea;
  if (info->off_ring + (uint32_t)CW * 2u * entry > kSmemLimit) return RWKVQ_EUNSUPPORTED;
  int depth = (int)((kSmemLimit - info->off_ring) / ((uint32_t)CW * entry));
  if (depth > 6) depth = 6;   // cp_async_wait_pending counts up to six groups in flight
  info->depth = depth;
  info->smem_bytes = info->off_ring + (uint32_t)CW * (uint32_t)depth * entry;

  size_t off = 256;
  info->off_desc_off = off; off += round_up_sz((size_t)(P + 1) * 4, 256);
  info->off_init_post = off; off += round_up_sz((size_t)P * 4, 256);
  info->off_descs = off; off += round_up_sz(descs.size() * sizeof(PhaseDesc), 256);
  info->off_flags = off; off += round_up_sz((size_t)P * 4, 256);
  info->off_gcnt = off; off += round_up_sz((size_t)gslots * 4, 256);
  info->off_gpart = off; off += round_up_sz((size_t)gslots * info->slot_floats * 4, 256);
  info->total_bytes = off;
  if (out) {
    out->assign(info->off_gpart, 0);     // the slab sums need no initial value
    memcpy(out->data() + info->off_desc_off, desc_off.data(), (size_t)(P + 1) * 4);
    memcpy(out->data() + info->off_init_post, init_post.data(), (size_t)P * 4);
    memcpy(out->data() + info->off_descs, descs.data(), descs.size() * sizeof(PhaseDesc));
  }
  return RWKVQ_OK;
}

static int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
  return sms;
}

static size_t trace_bytes_of(const PlanInfo& info) {
  return ((size_t)info.P * (size_t)(info.CW + 2) * kTraceSlots + (size_t)info.P * kTraceStages * 4) * sizeof(unsigned long long);
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
  info.abort_epoch = abort_epoch();   // the image just copied holds zeroed flags and counters
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  g_plans[plan_dev] = info;
  return RWKVQ_OK;
}

rwkvq_status rwkvq_step_run(const void* plan_dev, size_t plan_bytes, void* stream) {
  if (!plan_dev) return RWKVQ_EINVAL;
  PlanInfo info;
  bool clear_flags = false;
  {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    auto it = g_plans.find(plan_dev);
    if (it == g_plans.end()) return RWKVQ_EINVAL;   // not a plan written by rwkvq_step_plan in this process
    if (plan_bytes < it->second.total_bytes) return RWKVQ_ENOMEM;
    // The flags only ever grow: a run starts with every flag at (runs so far) * stages, so a launch
    // needs no clearing pass.  A run that gave up leaves them (and the slab counters) uneven; start
    // over after one.
    const unsigned epoch = abort_epoch();
    if (it->second.abort_epoch != epoch) { it->second.abort_epoch = epoch; it->second.runs = 0; clear_flags = true; }
    it->second.runs += 1;
    info = it->second;
  }
  const uint8_t* p = static_cast<const uint8_t*>(plan_dev);
  uint8_t* pw = const_cast<uint8_t*>(p);
  StepArgs a;
  a.descs = reinterpret_cast<const PhaseDesc*>(p + info.off_descs);
  a.desc_off = reinterpret_cast<const uint32_t*>(p + info.off_desc_off);
  a.init_post = reinterpret_cast<const uint32_t*>(p + info.off_init_post);
  a.flags = reinterpret_cast<unsigned*>(pw + info.off_flags);
  a.base = (info.runs - 1u) * (unsigned)info.n_stages;
  a.status = device_status_ptr();
  if (!a.status) return RWKVQ_ECUDA;
  a.poll_limit = info.poll_limit; a.wait_skew = info.wait_skew;
  a.B = info.B; a.nbp = (info.B + 1) & ~1; a.depth = info.depth;
  a.entry_bytes = info.entry_bytes; a.slot_floats = info.slot_floats;
  a.off_hq = info.off_hq; a.off_partial = info.off_partial; a.off_x = info.off_x; a.off_ring = info.off_ring;
  a.gcnt = reinterpret_cast<unsigned*>(pw + info.off_gcnt);
  a.gpart = reinterpret_cast<float*>(pw + info.off_gpart);
  a.trace = static_cast<unsigned long long*>(info.trace_dev);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaSuccess;
  if (clear_flags) {
    e = cudaMemsetAsync(a.flags, 0, info.off_gpart - info.off_flags, s);
    if (e != cudaSuccess) return cuda_status(e);
  }
  const void* fn;
  if (info.trace_dev) fn = info.NB == 1 ? (const void*)step_kernel<1, kConsumerWarps, true> : (const void*)step_kernel<2, kConsumerWarps, true>;
  else fn = info.NB == 1 ? (const void*)step_kernel<1, kConsumerWarps, false> : (const void*)step_kernel<2, kConsumerWarps, false>;
  e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)info.smem_bytes);
  if (e != cudaSuccess) return cuda_status(e);
  void* params[] = {&a};
  // Cooperative launch: all CTAs must be resident at once because they meet at the stage barrier.
  e = cudaLaunchCooperativeKernel(fn, dim3(info.P), dim3((info.CW + 2) * 32), params, info.smem_bytes, s);
  if (e != cudaSuccess) {   // this run will never report: have the next one clear the flags
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    auto it = g_plans.find(plan_dev);
    if (it != g_plans.end()) it->second.abort_epoch = abort_epoch() - 1u;
  }
  return cuda_status(e);
}

rwkvq_status rwkvq_step_plan_release(const void* plan_dev) {
  if (!plan_dev) return RWKVQ_EINVAL;
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  return g_plans.erase(plan_dev) ? RWKVQ_OK : RWKVQ_EINVAL;
}

rwkvq_status rwkvq_step_set_wait(const void* plan_dev, uint32_t poll_limit, uint32_t wait_skew) {
  if (!plan_dev) return RWKVQ_EINVAL;
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  auto it = g_plans.find(plan_dev);
  if (it == g_plans.end()) return RWKVQ_EINVAL;
  it->second.poll_limit = poll_limit ? poll_limit : kDefaultPollLimit;
  it->second.wait_skew = wait_skew;
  return RWKVQ_OK;
}

size_t rwkvq_step_trace_bytes(const void* plan_dev) {
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  auto it = g_plans.find(plan_dev);
  if (it == g_plans.end()) return 0;
  return trace_bytes_of(it->second);
}

rwkvq_status rwkvq_step_trace(const void* plan_dev, void* trace_dev, size_t trace_bytes) {
  if (!plan_dev) return RWKVQ_EINVAL;
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  auto it = g_plans.find(plan_dev);
  if (it == g_plans.end()) return RWKVQ_EINVAL;
  if (trace_dev) {
    if (((uintptr_t)trace_dev & 7u) != 0) return RWKVQ_EALIGN;
    if (trace_bytes < trace_bytes_of(it->second)) return RWKVQ_ENOMEM;
  }
  it->second.trace_dev = trace_dev;
  return RWKVQ_OK;
}

rwkvq_status rwkvq_step_plan_cover(const rwkvq_gemv_op* ops, int n_ops, int B, int n_ctas, uint32_t* counts_host,
                                   size_t n_counts, uint32_t* cta_items_host) {
  if (!counts_host || n_ctas <= 0) return RWKVQ_EINVAL;
  PlanInfo info;
  std::vector<uint8_t> image;
  rwkvq_status st = build_plan(ops, n_ops, B, n_ctas, &image, &info);
  if (st != RWKVQ_OK) return st;
  // cell of (product, 16-row slice, column tile) in counts_host
  std::vector<size_t> base(n_ops + 1, 0);
  for (int i = 0; i < n_ops; ++i) base[i + 1] = base[i] + (size_t)(ops[i].W_desc.oc / 16) * (size_t)(ops[i].W_desc.ic_pad / 256);
  if (n_counts < base[n_ops]) return RWKVQ_ENOMEM;
  std::unordered_map<uint64_t, int> op_of_y;
  for (int i = 0; i < n_ops; ++i) op_of_y[(uint64_t)(uintptr_t)ops[i].y_dev] = i;
  const uint32_t* desc_off = reinterpret_cast<const uint32_t*>(image.data() + info.off_desc_off);
  const PhaseDesc* descs = reinterpret_cast<const PhaseDesc*>(image.data() + info.off_descs);
  const int n_stages = info.n_stages;
  for (int c = 0; c < n_ctas; ++c) {
    uint32_t items = 0;
    bool in_group = false;
    uint32_t area = 0;
    for (uint32_t k = desc_off[c]; k < desc_off[c + 1]; ++k) {
      const PhaseDesc& d = descs[k];
      if ((d.kind_flags & 15u) != DK_PHASE) continue;
      auto it = op_of_y.find(d.y);
      if (it == op_of_y.end()) return RWKVQ_EINVAL;     // the walk needs distinct output buffers
      const int o = it->second;
      const uint32_t KT = d.KT, N = d.S * d.T, ks = d.ks_part & 0xFFFFu, part = d.ks_part >> 16;
      if (KT != (uint32_t)ops[o].W_desc.ic_pad / 256u || d.T * ks != KT || part >= ks || d.kt0 != part * d.T) return RWKVQ_EINVAL;
      // staging groups: every phase inside exactly one, the first phase of a stage opens one, segments disjoint
      if (d.kind_flags & DF_GROUP) { if (in_group) return RWKVQ_EINVAL; in_group = true; area = 0; }
      if (!in_group || ((d.kind_flags & DF_FIRST) && !(d.kind_flags & DF_GROUP))) return RWKVQ_EINVAL;
      if (d.xoff != area) return RWKVQ_EINVAL;
      area += xseg_bytes(B, (B + 1) & ~1, d.T * 256u, ops[o].W_desc.method == RWKVQ_SQ);
      if (info.off_x + area > info.off_ring) return RWKVQ_EINVAL;
      if (d.kind_flags & DF_GLAST) in_group = false;
      if ((d.kind_flags & DF_LAST) && in_group) return RWKVQ_EINVAL;
      // the walk of producer_role: every warp's share of the S x T grid
      for (uint32_t w = 0; w < (uint32_t)info.CW; ++w) {
        uint32_t i0, i1;
        item_range<kConsumerWarps>(N, w, i0, i1);
        for (uint32_t i = i0; i < i1; ++i) {
          const uint32_t sl = i / d.T, tt = i - sl * d.T;
          const uint32_t slice = d.row0 / 16u + sl, kt = d.kt0 + tt;
          if (slice >= (uint32_t)ops[o].W_desc.oc / 16u || kt >= KT) return RWKVQ_EINVAL;
          counts_host[base[o] + (size_t)slice * KT + kt] += 1u;
          ++items;
        }
      }
      if (ks > 1u && d.gslot0 + d.S * ks > info.gslots) return RWKVQ_EINVAL;
      if (d.post_value > (uint32_t)n_stages || d.post_value <= d.stage) return RWKVQ_EINVAL;
    }
    if (cta_items_host) cta_items_host[c] = items;
  }
  return RWKVQ_OK;
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
