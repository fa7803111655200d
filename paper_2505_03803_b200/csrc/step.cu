// A whole decode step as one persistent launch.
//
// Decode at batch 1..16 reads every packed weight once and does almost no arithmetic per byte
// (the paper's compute-to-memory argument, Section 1 and Appendix A.3), and one projection of a
// 7B-class layer is only a few microseconds of HBM time.  The step is therefore ONE cooperative
// kernel with one CTA per SM, built around three ideas:
//
//   * Weights never depend on activations, so each consumer warp owns a private ring of
//     shared-memory entries that a producer warp keeps full with bulk asynchronous copies
//     (cp.async.bulk + mbarrier transaction counts), one 16-row x 256-column record per entry,
//     running ahead across products and across stage boundaries.  HBM keeps streaming while the
//     CTAs synchronise.
//   * Every 16-row slice of a product (its whole K range) belongs to ONE CTA.  The slice's records
//     are dealt to the CTA's consumer warps in contiguous runs along K; a warp accumulates a run in
//     registers (m16n8k16 tensor-core steps, fp32), writes one partial per run to shared memory,
//     and the last warp to finish a slice adds the partials in warp order and stores y with plain
//     stores.  No atomics on outputs, no clearing pass, bit-reproducible results.
//   * The stage order ("every product of stage s is complete before any activation of stage s+1 is
//     read") is a flag-array grid barrier: a CTA publishes the number of stages it has completed
//     with one release store to its own word, and one auxiliary warp per CTA polls all words.
//
// Inputs.  With up to three batch rows every CTA mixes the activations it needs itself, right after
// the barrier opens (x_mix = x + (x_prev - x) (.) mu_hat, Appendix A.1 Eq. 20; x_prev and mu_hat
// are fetched before the barrier opens).  With larger batches all CTAs together compute the
// stage's x_mix once into a scratch area (a second flag barrier per stage) and every CTA then
// streams the windows of x_mix it needs into shared memory with bulk copies.
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

enum { DK_PHASE = 0, DK_PREPASS = 1, DK_END = 2 };
enum : uint32_t { DF_FIRST = 1u << 8, DF_LAST = 1u << 9, DF_MU = 1u << 10, DF_SUMS = 1u << 11, DF_SYNC = 1u << 12 };
// kind in bits 0..3, format (FMT_*) in bits 4..5 of kind_flags

// One phase of a CTA: slices [row0/16, row0/16 + S) of one product, all KT column tiles, walked in
// n_win windows of T tiles.  Item i of a window's S x T grid (slice-major) goes to consumer warp w
// with  w*N/CW <= i < (w+1)*N/CW  (N = S*T), the same split in every window, so a warp keeps the
// accumulators of at most two slices across the windows of a phase.
struct PhaseDesc {           // 128 bytes
  uint32_t kind_flags, stage;
  uint64_t src;              // payload of the product's image
  uint64_t cb;               // VQ: codebooks of the image
  uint64_t y;                // float y[B][oc]
  uint32_t oc, row0;         // rows of the product; first row of the phase
  uint32_t S, KT;            // DK_PREPASS: first product of the stage in the pre-pass table, count
  uint32_t T, n_win;         // DK_PREPASS: this CTA's share [T, n_win) of the stage's group list
  uint32_t xoff, xstride;    // bytes: the product's input rows inside the input area (window-relative when n_win > 1)
  uint32_t gsoff, cnt_base;  // bytes: group sums; first slice counter of the phase
  uint32_t win_seq0;         // number of this CTA's windows before this phase
  uint32_t items_end;        // items this CTA has consumed when the phase's STAGE is complete (mod 2^32)
  uint32_t post_value;       // stages to report complete at that point
  uint32_t ic;
  uint64_t x, xprev, mu, mu_aux;   // direct mode: the caller's inputs.  pre-pass mode: x, xprev = offsets of x_mix, sums in the scratch
  uint16_t mu_bits, mu_entries;
  uint32_t slot_set;         // which set of partial-sum slots the phase uses (phases of one stage alternate)
};
static_assert(sizeof(PhaseDesc) == 128, "phase descriptor size");

// One product's share of a stage's pre-pass: where its inputs are and where x_mix (fp16 rows of
// ic_pad columns, zero beyond ic) and the per-group sums ([group][3][nbp] floats) go.
struct StepMixOp {           // 64 bytes
  uint64_t x, xprev, mu, mu_aux, dst_x, dst_sums;
  uint32_t ic, ic_pad;
  uint16_t mu_bits, mu_entries, sums, pad;
};
static_assert(sizeof(StepMixOp) == 64, "pre-pass descriptor size");

// item header flags (word 2 of the 32-byte header the producer writes in front of every record)
enum : uint32_t {
  IF_ZERO = 1u << 2, IF_FLUSH = 1u << 3, IF_SWAP = 1u << 4, IF_XWAIT = 1u << 5,
  IF_RSELF = 1u << 29, IF_RFIRST = 1u << 30
};

constexpr int kConsumerWarps = 20;   // per CTA, plus one producer and one auxiliary warp
constexpr int kMaxCW = 24, kMaxDepth = 8, kHeaderRing = 8, kDescRing = 32, kMaxXBuf = 4, kCnt = 128;
constexpr uint32_t kCtrlBytes = 4096, kDescBytes = kDescRing * 128;
constexpr uint32_t kSmemLimit = 232448;  // 227 KB
constexpr uint32_t kDefaultPollLimit = 1u << 22;
enum { MODE_DIRECT = 0, MODE_PREPASS = 1 };

struct StepArgs {
  const PhaseDesc* descs;
  const uint32_t* desc_off;   // [P+1]
  const uint32_t* init_post;  // [P] stages a CTA may report complete before it has consumed anything
  unsigned* flags;            // [P] stages completed by each CTA, summed over all runs
  unsigned* flags2;           // [P] pre-passes completed
  unsigned base;              // value of every flag when this run starts
  int* status;
  uint32_t poll_limit;
  unsigned wait_skew;         // added to every barrier target (0; a test sets it to make the waits run out)
  int B, nbp, depth;
  uint32_t entry_bytes, slot_floats;
  uint32_t off_hq, off_partial, off_x, off_ring;
  uint32_t xwin_bytes, nxb;
  const StepMixOp* mixops;
  uint8_t* scratch;
  unsigned long long* trace;   // rwkvq_step_trace: per-warp counters, else NULL
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
// The hint lets the hardware park the thread for up to that many nanoseconds (it is woken when
// the phase completes), so that waiting warps do not compete for issue slots with computing ones.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(2000u) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Packed weights are read exactly once per step: they are marked evict-first so that streaming
// them does not push the activations, the plan and the outputs out of L2.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_g2s_plain(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ unsigned ld_relaxed_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_gpu(unsigned* p, unsigned v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
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
  uint64_t full[kMaxCW * kMaxDepth];   // per consumer warp and ring entry: the entry's copies have landed
  uint64_t xfull[kMaxXBuf];
  uint64_t open;               // the aux warp arrives once per stage this CTA takes part in
  uint32_t win_done[kMaxXBuf]; // items that have finished reading the window in each buffer
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

struct Env {
  const StepArgs& a;
  uint8_t* smem;
  Ctrl* ctrl;
  volatile int* abortp;
};

// Optional per-warp cycle accounting (rwkvq_step_trace): kTraceSlots 64-bit counters per warp,
// (CW + 2) warps per CTA.  Compiled into separate kernel instances, so the ordinary launch carries
// none of it.
constexpr int kTraceSlots = 16;
enum { TR_WAIT_FULL = 0, TR_WAIT_OPEN, TR_PRE, TR_POST, TR_ITEMS, TR_FLUSH, TR_NITEMS, TR_TOTAL, TR_WAIT_DESC, TR_WAIT_X,
       TR_P_ITER = 0, TR_P_ISSUED, TR_P_TOTAL, TR_P_IDLE, TR_P_WORK,
       TR_A_WAIT = 0, TR_A_POLLS, TR_A_REFILL, TR_A_TOTAL, TR_A_WIN };
template <bool TRACE>
struct Tracer {
  unsigned long long v[TRACE ? kTraceSlots : 1];
  __device__ __forceinline__ Tracer() {
    if constexpr (TRACE) for (int k = 0; k < kTraceSlots; ++k) v[k] = 0ull;
  }
  __device__ __forceinline__ long long now() const { if constexpr (TRACE) return clock64(); else return 0; }
  __device__ __forceinline__ void add(int slot, long long t0) { if constexpr (TRACE) v[slot] += (unsigned long long)(clock64() - t0); }
  __device__ __forceinline__ void count(int slot, unsigned n = 1u) { if constexpr (TRACE) v[slot] += n; }
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

// The share [i0, i1) of a window's N = S*T items that consumer warp w of CW owns.
template <int CW>
__host__ __device__ __forceinline__ void item_range(uint32_t N, uint32_t w, uint32_t& i0, uint32_t& i1) {
  if (N >= (uint32_t)CW) { i0 = w * N / (uint32_t)CW; i1 = (w + 1u) * N / (uint32_t)CW; }
  else { i0 = w < N ? w : N; i1 = w + 1u < N ? w + 1u : N; }
}

// ---- producer: one lane per consumer warp ---------------------------------------------------------
//
// Lane w walks the CTA's phases and writes, for every item of warp w in consumption order, a
// 64-byte item header into warp w's header ring: where the record (and, for VQ, its codebook) is in
// global memory, where its inputs are in shared memory, what to do with the accumulators and, on
// the last item of a run, where the outputs go.  It runs a few items ahead of the consumer, which
// issues the copies itself; all the index arithmetic of the schedule stays off the consumer warps.
//   q0 = { xoff/16 | gsoff/16 << 16, flags, xstride/16, codebook bytes }
//   q1 = { record address, codebook address }       q2 = { y, oc, first row }   (q2: IF_FLUSH only)
template <int CW, bool TRACE>
__device__ void producer_role(const Env& e) {
  const StepArgs& a = e.a;
  Tracer<TRACE> tr;
  const long long t_begin = tr.now();
  const uint32_t w = threadIdx.x & 31u;
  const bool active = w < (uint32_t)CW;
  uint8_t* hq = e.smem + a.off_hq + (size_t)w * kHeaderRing * 64u;
  uint32_t p = 0;              // descriptor this lane works on
  bool have = false, done = !active;
  // current phase
  uint32_t kf = 0, KT = 0, T = 0, n_win = 0, N = 0, i0 = 0, i1 = 0, rec_bytes = 0, cb_bytes = 0;
  uint32_t j = 0, i = 0, sl = 0, tt = 0, sl0 = 0, tt0 = 0, cur_set = 0;
  uint32_t n = 0;              // headers written
  uint32_t idle = 0, last_pmin = 0;
  while (true) {
    bool progress = false;
    tr.count(TR_P_ITER);
    const long long t_it = tr.now();
    if (!done && !have) {
      if ((int)(ld_acquire_cta(&e.ctrl->desc_hi) - p) > 0) {
        const PhaseDesc* d = desc_slot(e, p);
        kf = d->kind_flags;
        const uint32_t kind = kf & 15u;
        progress = true;
        if (kind == DK_END) done = true;
        else if (kind == DK_PREPASS) ++p;
        else {
          KT = d->KT; T = d->T; n_win = d->n_win; N = d->S * T;
          item_range<CW>(N, w, i0, i1);
          if (i0 == i1) ++p;
          else {
            have = true;
            const uint32_t fmt = (kf >> 4) & 3u;
            rec_bytes = fmt == FMT_SQ3 ? (uint32_t)RWKVQ_SQ_RECORD_BYTES : fmt == FMT_VQ6 ? 1536u : 2048u;
            cb_bytes = fmt == FMT_SQ3 ? 0u : fmt == FMT_VQ6 ? 256u : 1024u;
            sl0 = i0 / T; tt0 = i0 - sl0 * T;
            j = 0; i = i0; sl = sl0; tt = tt0; cur_set = 0;
          }
        }
      }
    } else if (!done) {
      if (n - ld_acquire_cta(&e.ctrl->hq_tail[w]) < (uint32_t)kHeaderRing) {
        progress = true;
        const PhaseDesc* d = desc_slot(e, p);
        const uint32_t fmt = (kf >> 4) & 3u;
        const uint32_t kt = j * T + tt;
        const uint32_t row = d->row0 + 16u * sl;
        const uint64_t src = d->src + ((uint64_t)(row >> 7) * KT + kt) * (8u * rec_bytes) + (uint64_t)((row >> 4) & 7u) * rec_bytes;
        const uint64_t cbs = cb_bytes ? d->cb + ((uint64_t)(row >> 8) * KT + kt) * cb_bytes : 0ull;
        const uint32_t nbp = (uint32_t)a.nbp;
        const uint32_t tcol = n_win > 1u ? tt : kt;         // tile position inside the resident input rows
        uint32_t xo = d->xoff + tcol * 512u, go = d->gsoff + tcol * (2u * 3u * nbp * 4u);
        uint32_t flags = fmt;
        if (a.nxb) {                                        // pre-pass mode: the inputs sit in a copied window
          const uint32_t seq = d->win_seq0 + j, buf = seq % a.nxb;
          xo += buf * a.xwin_bytes; go += buf * a.xwin_bytes;
          flags |= IF_XWAIT | (buf << 6) | (((seq / a.nxb) & 1u) << 8);
          if (n_win > 1u) {
            const uint32_t r = sl != sl0 ? 1u : 0u;
            if (r != cur_set) { flags |= IF_SWAP; cur_set = r; }
          }
        }
        const bool run_first = (i == i0 || tt == 0u), run_last = (i + 1u == i1 || tt + 1u == T);
        if (j == 0u && run_first) flags |= IF_ZERO;
        uint4 q2 = make_uint4(0u, 0u, 0u, 0u);
        if (j + 1u == n_win && run_last) {
          // the slice ends here for this warp: who else contributes, and where the rows go
          const uint32_t lo = sl * T, hi = lo + T;
          uint32_t wlo, whi;
          if (N >= (uint32_t)CW) { wlo = ((lo + 1u) * (uint32_t)CW + N - 1u) / N - 1u; whi = (hi * (uint32_t)CW + N - 1u) / N - 1u; }
          else { wlo = lo; whi = hi - 1u; }
          uint32_t f0, f1;
          item_range<CW>(N, wlo, f0, f1);
          flags |= IF_FLUSH | (((d->cnt_base + sl) & (uint32_t)(kCnt - 1)) << 9) | ((whi - wlo + 1u) << 16) | (wlo << 24);
          if (sl != sl0) flags |= IF_RSELF;
          if (f0 < lo) flags |= IF_RFIRST;
          q2 = make_uint4((uint32_t)d->y, (uint32_t)(d->y >> 32), d->oc, row);
        }
        uint4* h = reinterpret_cast<uint4*>(hq + (size_t)(n % (uint32_t)kHeaderRing) * 64u);
        h[0] = make_uint4((xo >> 4) | ((go >> 4) << 16), flags, d->xstride >> 4, cb_bytes);
        h[1] = make_uint4((uint32_t)src, (uint32_t)(src >> 32), (uint32_t)cbs, (uint32_t)(cbs >> 32));
        h[2] = q2;
        ++n;
        st_release_cta(&e.ctrl->hq_head[w], n);
        tr.count(TR_P_ISSUED);
        // next item of this warp
        ++i; ++tt;
        if (tt == T) { tt = 0; ++sl; }
        if (i == i1) {
          i = i0; sl = sl0; tt = tt0;
          if (++j == n_win) { have = false; ++p; }
        }
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
  // every load is issued before the first result is looked at: one round trip per poll
  unsigned behind = 0u;
  for (int c = lane; c < P; c += 32) behind |= (ld_relaxed_gpu(flags + c) - target) >> 31;
  return __all_sync(0xFFFFFFFFu, behind == 0u);
}
__device__ __forceinline__ bool flags_wait(const Env& e, const unsigned* flags, unsigned target, int lane) {
  const int P = (int)gridDim.x;
  for (uint32_t it = 0; it < (e.a.poll_limit << 2); ++it) {
    if (flags_reached(flags, P, target, lane)) { fence_gpu(); return true; }
    if ((it & 7u) == 7u && *e.abortp) return false;
  }
  if (lane == 0) give_up(e);
  return false;
}

// ---- auxiliary warp: descriptor ring, barrier detection, input windows ----------------------------
template <int MODE, bool TRACE>
__device__ void aux_role(const Env& e) {
  const StepArgs& a = e.a;
  const int lane = threadIdx.x & 31;
  Tracer<TRACE> tr;
  const long long t_begin = tr.now();
  const uint32_t d0 = a.desc_off[blockIdx.x], n_desc = a.desc_off[blockIdx.x + 1] - d0;
  uint32_t hi = 0;
  auto refill = [&]() {
    // copy descriptors into the ring as far as the consumers' progress allows, four per pass
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
  uint32_t win_expect[kMaxXBuf] = {0u, 0u, 0u, 0u};
  for (uint32_t p = 0; p < n_desc; ++p) {
    if (p >= hi) {
      // the ring is full of descriptors the consumers still need: wait for them to move on
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
    const uint32_t kf = d->kind_flags, kind = kf & 15u;
    if (kind == DK_END) break;
    const uint32_t stage = d->stage;
    if (kind == DK_PREPASS || (MODE == MODE_DIRECT && (kf & DF_FIRST))) {
      // the stage may start once every CTA has completed all earlier stages
      const long long t0 = tr.now();
      if (stage > 0u && !flags_wait(e, a.flags, a.base + stage + a.wait_skew, lane)) return;
      tr.add(TR_A_WAIT, t0); tr.count(TR_A_POLLS);
      __syncwarp();
      if (lane == 0) mbar_arrive(&e.ctrl->open);
    }
    if (MODE == MODE_PREPASS) {
      if (kind == DK_PREPASS) {
        if (!flags_wait(e, a.flags2, a.base + stage + 1u + a.wait_skew, lane)) return;
      } else {
        // stream this phase's input windows: B rows of T tiles and the block of group sums each
        const uint32_t T = d->T, n_win = d->n_win, items = d->S * T;
        const uint32_t row_bytes = T * 512u;
        const uint32_t sums_bytes = (kf & DF_SUMS) ? T * 2u * 3u * (uint32_t)a.nbp * 4u : 0u;
        const uint32_t pitch = d->ic;                       // bytes between batch rows of x_mix in the scratch
        for (uint32_t j = 0; j < n_win; ++j) {
          const uint32_t seq = d->win_seq0 + j, buf = seq % a.nxb;
          bool ok = false;
          for (uint32_t it = 0; it < (a.poll_limit << 4); ++it) {
            if (ld_acquire_cta(&e.ctrl->win_done[buf]) == win_expect[buf]) { ok = true; break; }
            if ((it & 63u) == 63u && *e.abortp) break;
            __nanosleep(64);
          }
          if (!ok) { if (lane == 0 && !*e.abortp) give_up(e); return; }
          win_expect[buf] = items;
          __syncwarp();
          if (lane == 0) {
            st_release_cta(&e.ctrl->win_done[buf], 0u);
            // what other CTAs wrote with ordinary stores is read below by the copy engine
            asm volatile("fence.proxy.async;" ::: "memory");
            mbar_arrive_expect_tx(&e.ctrl->xfull[buf], (uint32_t)a.B * row_bytes + sums_bytes);
          }
          __syncwarp();
          const uint32_t dst = smem_u32(e.smem + a.off_x) + buf * a.xwin_bytes;
          const uint32_t bar = smem_u32(&e.ctrl->xfull[buf]);
          if (lane < a.B)
            bulk_g2s_plain(dst + d->xoff + (uint32_t)lane * d->xstride,
                           a.scratch + d->x + (size_t)lane * pitch + (size_t)j * row_bytes, row_bytes, bar);
          else if (lane == a.B && sums_bytes)
            bulk_g2s_plain(dst + d->gsoff, a.scratch + d->xprev + (size_t)j * sums_bytes, sums_bytes, bar);
        }
      }
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

// ---- consumer warps ---------------------------------------------------------------------------------

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

// This CTA's share of a stage's pre-pass.  A half-warp takes one (product, batch row, 128-column
// group) at a time: it loads x (and x_prev, and decodes mu_hat), mixes, rounds to fp16, stores the
// 128 values to the product's pre-pass rows and reduces the three sums of the group with shuffles.
template <int CW>
__device__ void prepass_share(const StepArgs& a, const PhaseDesc* d) {
  const int tid = threadIdx.x, lane = tid & 31, l16 = lane & 15;
  const uint32_t lo = d->T, hi = d->n_win;
  const StepMixOp* ops = a.mixops + d->S;
  const int n_ops = (int)d->KT;
  const int nbp = a.nbp;
  for (uint32_t g0 = lo + 2u * (uint32_t)(tid >> 5); g0 < hi; g0 += 2u * (uint32_t)CW) {
    const uint32_t gi = g0 + (uint32_t)(lane >> 4);
    const bool valid = gi < hi;
    uint32_t r = valid ? gi : lo;
    int k = 0;
    uint32_t icp = __ldg(&ops[0].ic_pad);
    while (k + 1 < n_ops && r >= (uint32_t)a.B * (icp >> 7)) { r -= (uint32_t)a.B * (icp >> 7); ++k; icp = __ldg(&ops[k].ic_pad); }
    const StepMixOp op = ops[k];
    const uint32_t ng = op.ic_pad >> 7;
    const int b = (int)(r / ng), grp = (int)(r % ng);
    const int col = grp * 128 + l16 * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (col < (int)op.ic) {
      v = __ldcg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(op.x) + (size_t)b * op.ic + col));
      if (op.mu) {
        const uint4 pr = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(op.xprev) + (size_t)b * op.ic + col));
        const uint4 m = mu_vector(reinterpret_cast<const uint8_t*>(op.mu), reinterpret_cast<const uint8_t*>(op.mu_aux), op.mu_bits, col);
        v.x = mix2(v.x, pr.x, m.x); v.y = mix2(v.y, pr.y, m.y); v.z = mix2(v.z, pr.z, m.z); v.w = mix2(v.w, pr.w, m.w);
      }
    }
    if (valid) *reinterpret_cast<uint4*>(reinterpret_cast<__half*>(a.scratch + op.dst_x) + (size_t)b * op.ic_pad + col) = v;
    float sx, nb0, nb1;
    group_sums(v, l16, sx, nb0, nb1);
    if (valid && l16 == 0 && op.sums) {
      float* gs = reinterpret_cast<float*>(a.scratch + op.dst_sums);
      gs[(grp * 3 + 0) * nbp + b] = sx;
      gs[(grp * 3 + 1) * nbp + b] = nb0;
      gs[(grp * 3 + 2) * nbp + b] = nb1;
    }
  }
}

// Direct mode: the consumer threads of a CTA mix the inputs of every phase [p0, p1) of a stage
// into the input area.  A thread owns 16-byte vectors (8 columns of one batch row) tid, tid + NT,
// ... of the concatenated phases; x_prev and mu_hat of its first two vectors are fetched BEFORE the
// grid barrier is awaited, so that only one round of loads of x, the mix and the sums follow it.
template <int CW>
struct DirectStager {
  static constexpr int NT = CW * 32, PRE = 2;
  uint4 xp[PRE], mh[PRE];

  // vector number v of the stage -> phase, batch row, vector within the row
  __device__ __forceinline__ static const PhaseDesc* locate(const Env& e, uint32_t p0, uint32_t p1, int B, uint32_t v, int& b, int& c8) {
    for (uint32_t p = p0; p < p1; ++p) {
      const PhaseDesc* d = desc_slot(e, p);
      const uint32_t nvr = d->KT * 32u, nv = (uint32_t)B * nvr;
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
      if (d && (d->kind_flags & DF_MU) && 8 * c8 < (int)d->ic) {
        xp[k] = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(d->xprev) + (size_t)b * d->ic + 8 * c8));
        mh[k] = mu_vector(reinterpret_cast<const uint8_t*>(d->mu), reinterpret_cast<const uint8_t*>(d->mu_aux), d->mu_bits, 8 * c8);
      }
    }
  }
  // Mix, round and store one vector; reduce the group's sums.  Called by whole warps.
  __device__ __forceinline__ static void finish_vector(const Env& e, const PhaseDesc* d, int b, int c8, bool pre, uint4 pr, uint4 m) {
    const int lane = threadIdx.x & 31, nbp = e.a.nbp;
    uint8_t* xarea = e.smem + e.a.off_x;
    const int col = 8 * c8;
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
  // every branch below is warp-uniform.
  __device__ __forceinline__ void after_barrier(const Env& e, uint32_t p0, uint32_t p1) {
#pragma unroll
    for (int k = 0; k < PRE; ++k) {
      int b = 0, c8 = 0;
      const PhaseDesc* d = locate(e, p0, p1, e.a.B, (uint32_t)(threadIdx.x + k * NT), b, c8);
      if (!d) return;
      finish_vector(e, d, b, c8, true, xp[k], mh[k]);
    }
    for (int k = PRE;; ++k) {
      int b = 0, c8 = 0;
      const PhaseDesc* d = locate(e, p0, p1, e.a.B, (uint32_t)(threadIdx.x + k * NT), b, c8);
      if (!d) return;
      finish_vector(e, d, b, c8, false, make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u));
    }
  }
};

// One 128-column group of an SQ record (16 rows) against the staged input:
//   acc[b][row] += s * ( sum_cols (q+bias) x  -  Bx_h  -  z * Sx )
// The tensor-core accumulators start at -Bx_h (the bias every extracted half carries, taken
// from the precomputed sums), so after the eight m16n8k16 steps only two FMAs per output remain.
// `w`: the group's six words; sz_lo / sz_hi: (s, z) fp16 pairs of rows g and g+8; xrow[n]: this
// lane's fragment pointer into batch block n at the group's first column; gs: this lane's pointer
// to the group's sums [3][nbp] (already offset by 8 * (lane & 3) bytes).
template <int NB>
__device__ __forceinline__ void sq_group(const uint32_t (&w)[6], uint32_t sz_lo, uint32_t sz_hi, const uint8_t* const (&xrow)[NB],
                                         const uint8_t* gs, uint32_t gstride, float (&acc)[NB][4]) {
  float c[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const float2 b0 = *reinterpret_cast<const float2*>(gs + gstride + n * 32);
    const float2 b1 = *reinterpret_cast<const float2*>(gs + 2 * gstride + n * 32);
    c[n][0] = b0.x; c[n][1] = b0.y; c[n][2] = b1.x; c[n][3] = b1.y;
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
        const uint2 bf = *reinterpret_cast<const uint2*>(xrow[n] + (4 * ti + m) * 32);
        mma_16816(c[n], afrag, bf.x, bf.y);
      }
    }
  }
  const uint32_t nlo = sz_lo ^ 0x80000000u, nhi = sz_hi ^ 0x80000000u;   // (s, -z)
  const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&nlo));
  const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&nhi));
#pragma unroll
  for (int n = 0; n < NB; ++n) {
    const float2 sx = *reinterpret_cast<const float2*>(gs + n * 32);
    acc[n][0] = fmaf(s0.x, fmaf(s0.y, sx.x, c[n][0]), acc[n][0]);
    acc[n][1] = fmaf(s0.x, fmaf(s0.y, sx.y, c[n][1]), acc[n][1]);
    acc[n][2] = fmaf(s1.x, fmaf(s1.y, sx.x, c[n][2]), acc[n][2]);
    acc[n][3] = fmaf(s1.x, fmaf(s1.y, sx.y, c[n][3]), acc[n][3]);
  }
}

// Eight tensor-core steps (HALF of a tile's columns) of a VQ record: every fragment register is one
// lookup in the tile's codebook, which sits behind the record in the ring entry.
template <int BITS, int NB, int HALF>
__device__ __forceinline__ void vq_half(const uint32_t (&w)[2 * BITS], const uint32_t* cb, const uint8_t* const (&xrow)[NB],
                                        float (&acc)[NB][4]) {
#pragma unroll
  for (int j = 8 * HALF; j < 8 * HALF + 8; ++j) {
    uint32_t afrag[4];
#pragma unroll
    for (int R = 0; R < 4; ++R) afrag[R] = cb[vq_index<BITS, 2 * BITS>(w, 4 * j + R)];
#pragma unroll
    for (int n = 0; n < NB; ++n) {
      const uint2 bf = *reinterpret_cast<const uint2*>(xrow[n] + j * 32);
      mma_16816(acc[n], afrag, bf.x, bf.y);
    }
  }
}

// 16-byte asynchronous copies global -> shared, tracked by an mbarrier: the copies a lane has
// issued arrive on the barrier when they have landed (the barrier is initialised to one arrival
// per lane).
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src, uint64_t policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_arrive(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

template <int NB, int MODE, int CW, bool TRACE>
__device__ void consumer_role(const Env& e) {
  const StepArgs& a = e.a;
  Tracer<TRACE> tr;
  const long long t_begin = tr.now();
  const int lane = threadIdx.x & 31;
  const uint32_t w = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const uint32_t depth = (uint32_t)a.depth;
  uint8_t* ring = e.smem + a.off_ring + (size_t)w * depth * a.entry_bytes;
  const uint32_t ring_s = smem_u32(ring);
  const uint8_t* hq = e.smem + a.off_hq + (size_t)w * kHeaderRing * 64u;
  uint64_t* full = e.ctrl->full + w * kMaxDepth;
  const uint8_t* xarea = e.smem + a.off_x;
  float* partial = reinterpret_cast<float*>(e.smem + a.off_partial);
  const uint32_t gstride = (uint32_t)a.nbp * 4u;
  // weights are read once per step: evict-first, so that they do not push the activations, the
  // plan and the outputs out of L2
  const uint64_t policy = policy_evict_first();
  int rowsel[NB];
#pragma unroll
  for (int n = 0; n < NB; ++n) rowsel[n] = min(8 * n + g, a.B - 1);
  float acc[NB][4], alt[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n)
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[n][k] = alt[n][k] = 0.f;
  uint32_t n_cons = 0, n_iss = 0;      // items consumed / copies issued, over the whole launch
  uint32_t slot = 0, round = 0;        // n_cons % depth, n_cons / depth
  uint32_t islot = 0;                  // n_iss % depth
  uint32_t opened = 0;                 // stages this CTA has taken part in
  uint32_t reported = 0;               // stages with items this warp has left
  bool dead = false, verdict = false;  // verdict: the role's barrier has already told everyone to leave
  DirectStager<CW> stager;

  // Issue the copies of item n_iss (record, and codebook behind it) into ring entry islot, if its
  // header has been written; the entry is free because the warp itself has consumed what was in it.
  auto issue_one = [&]() -> bool {
    if ((int)(ld_acquire_cta(&e.ctrl->hq_head[w]) - n_iss) <= 0) return false;
    const uint4* h = reinterpret_cast<const uint4*>(hq + (size_t)(n_iss % (uint32_t)kHeaderRing) * 64u);
    const uint32_t fl = h[0].y, cbb = h[0].w;
    const uint4 q1 = h[1];
    const uint8_t* src = reinterpret_cast<const uint8_t*>(((uint64_t)q1.y << 32) | q1.x);
    const uint32_t fmt = fl & 3u;
    const uint32_t rec16 = fmt == FMT_SQ3 ? (uint32_t)RWKVQ_SQ_RECORD_BYTES / 16u : fmt == FMT_VQ6 ? 96u : 128u;
    const uint32_t dst = ring_s + islot * a.entry_bytes;
    for (uint32_t c = (uint32_t)lane; c < rec16; c += 32u) cp_async16(dst + c * 16u, src + (size_t)c * 16u, policy);
    if (cbb) {
      const uint8_t* cbs = reinterpret_cast<const uint8_t*>(((uint64_t)q1.w << 32) | q1.z);
      for (uint32_t c = (uint32_t)lane; c < cbb / 16u; c += 32u) cp_async16(dst + (rec16 + c) * 16u, cbs + (size_t)c * 16u, policy);
    }
    cp_async_arrive(&full[islot]);
    ++n_iss; if (++islot == depth) islot = 0;
    return true;
  };

  for (uint32_t p = 0;; ++p) {
    {
      const long long t0 = tr.now();
      if (!dead && !wait_desc(e, p)) dead = true;
      tr.add(TR_WAIT_DESC, t0);
    }
    if (dead) break;
    const PhaseDesc* d = desc_slot(e, p);
    const uint32_t kf = d->kind_flags, kind = kf & 15u;
    if (kind == DK_END) break;
    // top up the weight ring before anything that may wait
    while (n_iss - n_cons < depth && issue_one()) {}
    if (kind == DK_PREPASS || (MODE == MODE_DIRECT && (kf & DF_FIRST))) {
      uint32_t p1 = p + 1;
      if (MODE == MODE_DIRECT) {
        while (true) {               // the stage's phases: p .. the one flagged last
          if (!wait_desc(e, p1 - 1)) { dead = true; break; }
          if (desc_slot(e, p1 - 1)->kind_flags & DF_LAST) break;
          ++p1;
        }
        const long long t0 = tr.now();
        if (!dead) stager.before_barrier(e, p, p1);
        tr.add(TR_PRE, t0);
      }
      {
        const long long t0 = tr.now();
        if (!dead && !mbar_wait(e, &e.ctrl->open, opened & 1u)) dead = true;
        tr.add(TR_WAIT_OPEN, t0);
      }
      ++opened;
      const long long t1 = tr.now();
      if (!dead) {
        if (MODE == MODE_DIRECT) stager.after_barrier(e, p, p1);
        else prepass_share<CW>(a, d);
      }
      // every consumer thread's stores precede the verdict; all leave together after a failure
      if (!named_bar_and(1, CW * 32, !dead)) { dead = true; verdict = true; break; }
      tr.add(TR_POST, t1);
      if (threadIdx.x == 0) {
        st_release_cta(&e.ctrl->desc_tail, p);
        if (MODE == MODE_PREPASS) { fence_gpu(); st_relaxed_gpu(a.flags2 + blockIdx.x, a.base + d->stage + 1u); }
      }
      if (kind == DK_PREPASS) continue;
    }
    // the phase reuses a set of partial-sum slots of an earlier phase of this stage: every warp must
    // have left that phase (its slices are then reduced and stored)
    if ((kf & DF_SYNC) && !named_bar_and(1, CW * 32, true)) { dead = true; verdict = true; break; }
    const uint32_t slot0 = d->slot_set * 2u * (uint32_t)CW;
    uint32_t i0, i1;
    item_range<CW>(d->S * d->T, w, i0, i1);
    const uint32_t n_my = (i1 - i0) * d->n_win;
    for (uint32_t it = 0; it < n_my; ++it) {
      const long long t_w = tr.now();
      while (n_iss - n_cons < depth && issue_one()) {}
      if (n_iss == n_cons) {
        // the header of this very item has not been written yet: wait for the producer lane (bounded)
        bool ok = false;
        for (uint32_t k = 0; k < (a.poll_limit << 4); ++k) {
          if (issue_one()) { ok = true; break; }
          if ((k & 63u) == 63u && *e.abortp) break;
          __nanosleep(32);
        }
        if (!ok) { if (!*e.abortp) give_up(e); dead = true; break; }
      }
      if (!mbar_wait(e, &full[slot], round & 1u)) { dead = true; break; }
      tr.add(TR_WAIT_FULL, t_w);
      const long long t_i = tr.now();
      tr.count(TR_NITEMS);
      const uint4* hdr = reinterpret_cast<const uint4*>(hq + (size_t)(n_cons % (uint32_t)kHeaderRing) * 64u);
      const uint4 ha = hdr[0];
      const uint32_t flags = ha.y;
      uint4 hb = make_uint4(0u, 0u, 0u, 0u);
      if (flags & IF_FLUSH) hb = hdr[2];
      __syncwarp();
      if (lane == 0) st_release_cta(&e.ctrl->hq_tail[w], n_cons + 1u);   // the header is in registers
      if (flags & IF_SWAP) {
#pragma unroll
        for (int n = 0; n < NB; ++n)
#pragma unroll
          for (int k = 0; k < 4; ++k) { const float tmp = acc[n][k]; acc[n][k] = alt[n][k]; alt[n][k] = tmp; }
      }
      if (flags & IF_ZERO) {
#pragma unroll
        for (int n = 0; n < NB; ++n)
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[n][k] = 0.f;
      }
      if (MODE == MODE_PREPASS) {
        const long long t_x = tr.now();
        if (!mbar_wait(e, &e.ctrl->xfull[(flags >> 6) & 3u], (flags >> 8) & 1u)) { dead = true; break; }
        tr.add(TR_WAIT_X, t_x);
      }
      const uint32_t xstride = ha.z << 4;
      const uint8_t* xt = xarea + ((ha.x & 0xFFFFu) << 4) + t * 8;
      const uint8_t* xrow[NB];
#pragma unroll
      for (int n = 0; n < NB; ++n) xrow[n] = xt + (size_t)rowsel[n] * xstride;
      const uint8_t* rec = ring + (size_t)slot * a.entry_bytes;
      const uint32_t fmt = flags & 3u;
      if (fmt == FMT_SQ3) {
        const uint4 p0 = *reinterpret_cast<const uint4*>(rec + lane * 16);
        const uint4 p1 = *reinterpret_cast<const uint4*>(rec + 512 + lane * 16);
        const uint4 p2 = *reinterpret_cast<const uint4*>(rec + 1024 + lane * 16);
        const uint4 sz = *reinterpret_cast<const uint4*>(rec + RWKVQ_SQ_CODE_BYTES + g * 16);
        // the record is in registers: once every lane has read its part, the entry is refilled
        __syncwarp();
        ++n_cons; if (++slot == depth) { slot = 0; ++round; }
        issue_one();
        const uint8_t* gs = xarea + ((ha.x >> 16) << 4) + t * 8;
        {
          const uint32_t w0[6] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y};
          sq_group<NB>(w0, sz.x, sz.z, xrow, gs, gstride, acc);
        }
        {
          const uint8_t* xr1[NB];
#pragma unroll
          for (int n = 0; n < NB; ++n) xr1[n] = xrow[n] + 256;
          const uint32_t w1[6] = {p1.z, p1.w, p2.x, p2.y, p2.z, p2.w};
          sq_group<NB>(w1, sz.y, sz.w, xr1, gs + 3 * gstride, gstride, acc);
        }
      } else {
        if (fmt == FMT_VQ6) {
          const uint32_t* cb = reinterpret_cast<const uint32_t*>(rec + 1536);
          uint32_t v[12];
          vq_half_words<6, 0>(rec, lane, v);
          vq_half_words<6, 1>(rec, lane, v);
          vq_half<6, NB, 0>(v, cb, xrow, acc);
          vq_half<6, NB, 1>(v, cb, xrow, acc);
        } else {
          const uint32_t* cb = reinterpret_cast<const uint32_t*>(rec + 2048);
          uint32_t v[16];
          vq_half_words<8, 0>(rec, lane, v);
          vq_half<8, NB, 0>(v, cb, xrow, acc);
          vq_half_words<8, 1>(rec, lane, v);
          vq_half<8, NB, 1>(v, cb, xrow, acc);
        }
        // the codebook is looked up in the entry until the last step
        __syncwarp();
        ++n_cons; if (++slot == depth) { slot = 0; ++round; }
        issue_one();
      }
      if (MODE == MODE_PREPASS) {
        __syncwarp();
        if (lane == 0) asm volatile("red.release.cta.shared::cta.add.u32 [%0], 1;" ::"r"(smem_u32(&e.ctrl->win_done[(flags >> 6) & 3u])) : "memory");
      }
      const long long t_f = tr.now();
      if (flags & IF_FLUSH) {
        float* y = reinterpret_cast<float*>(((uint64_t)hb.y << 32) | hb.x);
        const uint32_t oc = hb.z, row = hb.w;
        const uint32_t ncon = (flags >> 16) & 0xFFu;
        if (ncon == 1u) {
#pragma unroll
          for (int n = 0; n < NB; ++n)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int b = n * 8 + 2 * t + (k & 1);
              if (b < a.B) y[(size_t)b * oc + row + (uint32_t)g + 8u * (uint32_t)(k >> 1)] = acc[n][k];
            }
        } else {
          float* ps = partial + (size_t)(slot0 + 2u * w + ((flags >> 29) & 1u)) * a.slot_floats;
#pragma unroll
          for (int n = 0; n < NB; ++n)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int b = n * 8 + 2 * t + (k & 1);
              if (b < a.B) ps[b * 16 + g + 8 * (k >> 1)] = acc[n][k];
            }
          __syncwarp();
          uint32_t old = 0;
          uint32_t* cnt = &e.ctrl->cnt[(flags >> 9) & (uint32_t)(kCnt - 1)];
          if (lane == 0) old = smem_add_acq_rel(cnt, 1u);
          old = __shfl_sync(0xFFFFFFFFu, old, 0);
          __syncwarp();
          if (old + 1u == ncon) {
            // last of the slice's warps: add the partials in warp order, store the rows
            if (lane == 0) *cnt = 0u;
            const uint32_t wlo = (flags >> 24) & 31u, rfirst = (flags >> 30) & 1u;
            for (int el = lane; el < 16 * a.B; el += 32) {
              float sum = 0.f;
              for (uint32_t k = 0; k < ncon; ++k)
                sum += partial[(size_t)(slot0 + 2u * (wlo + k) + (k == 0u ? rfirst : 0u)) * a.slot_floats + el];
              y[(size_t)(el >> 4) * oc + row + (uint32_t)(el & 15)] = sum;
            }
          }
        }
      }
      tr.add(TR_FLUSH, t_f);
      tr.add(TR_ITEMS, t_i);
    }
    if (dead) break;
    if (kf & DF_LAST) {
      // This warp has left the stage.  The count is an acquire-release read-modify-write at CTA scope
      // and the publication a GPU-scope release by whoever reports last, so it is ordered after
      // everything every warp stored before reporting: block-level synchronisation followed by one
      // thread's release, the pattern of a cooperative grid barrier.
      __syncwarp();
      if (lane == 0) {
        const uint32_t old = smem_add_acq_rel(&e.ctrl->warps_done, 1u);
        if (old + 1u == (uint32_t)CW * (reported + 1u)) { fence_gpu(); st_relaxed_gpu(a.flags + blockIdx.x, a.base + d->post_value); }
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


template <int NB, int MODE, int CW, bool TRACE>
__global__ void __launch_bounds__((CW + 2) * 32, 1) step_kernel(const StepArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem);
  if (threadIdx.x == 0) {
    for (int k = 0; k < kMaxCW * kMaxDepth; ++k) mbar_init(&ctrl->full[k], 32);
    for (int k = 0; k < kMaxCW; ++k) { ctrl->hq_head[k] = 0u; ctrl->hq_tail[k] = 0u; }
    for (int k = 0; k < kMaxXBuf; ++k) { mbar_init(&ctrl->xfull[k], 1); ctrl->win_done[k] = 0u; }
    mbar_init(&ctrl->open, 1);
    ctrl->warps_done = 0u; ctrl->desc_hi = 0u; ctrl->desc_tail = 0u; ctrl->prod_tail = 0u; ctrl->abort_flag = 0;
    for (int k = 0; k < kCnt; ++k) ctrl->cnt[k] = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const Env e{a, smem, ctrl, &ctrl->abort_flag};
  const int warp = threadIdx.x >> 5;
  if (warp < CW) consumer_role<NB, MODE, CW, TRACE>(e);
  else if (warp == CW) producer_role<CW, TRACE>(e);
  else aux_role<MODE, TRACE>(e);
}

// ---- host planner --------------------------------------------------------------------------------

struct PlanInfo {
  int P, B, NB, CW, mode, depth, n_stages;
  unsigned runs;        // launches since the flags were last zero
  unsigned abort_epoch; // value of the abort epoch when the flags were last known good
  uint32_t poll_limit, wait_skew, n_sets;
  void* trace_dev;      // rwkvq_step_trace: where the next runs write their per-warp counters
  uint32_t entry_bytes, slot_floats, smem_bytes, off_hq, off_partial, off_x, off_ring, xwin_bytes, nxb;
  size_t off_desc_off, off_init_post, off_descs, off_flags, off_flags2, off_mixops, off_scratch, total_bytes;
  uint32_t n_descs;
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

// Input-area footprint of one product held whole (direct mode): B rows of ic_pad fp16 values plus 32
// bytes of padding each (the 8-byte fragment loads of a half-warp then hit 16 distinct bank
// pairs), the group sums, and 64 bytes of slack that lanes of batch columns which do not exist
// read (and discard).
static uint32_t xrows_bytes(int B, uint32_t cols) { return (uint32_t)B * (cols * 2u + 32u); }
static uint32_t xsums_bytes(int nbp, uint32_t cols, bool sums) { return sums ? (cols / 128u) * 3u * (uint32_t)nbp * 4u + 64u : 0u; }

struct CtaPhase {
  int op;
  uint32_t row0, S;
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

  // 1. deal every stage's 16-row slices to the CTAs: contiguous in (product, row) order, balanced
  //    by cost (records x a weight per format: what a record costs a consumer warp)
  std::vector<std::vector<std::vector<CtaPhase>>> deal(n_stages, std::vector<std::vector<CtaPhase>>(P));
  for (int s = 0; s < n_stages; ++s) {
    uint64_t total = 0;
    auto slice_cost = [&](int o) -> uint64_t {
      const rwkvq_desc& d = ops[o].W_desc;
      const uint64_t wgt = d.method == RWKVQ_SQ ? 20u : d.bits == 8 ? 40u : 36u;
      return (uint64_t)(d.ic_pad / 256) * wgt;
    };
    for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) total += slice_cost(o) * (uint64_t)(ops[o].W_desc.oc / 16);
    uint64_t run = 0;
    const int rot = (int)(((uint64_t)s * 37u) % (uint64_t)P);   // idle CTAs of small stages are not always the same SMs
    for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) {
      const uint64_t c1 = slice_cost(o);
      const int ns = ops[o].W_desc.oc / 16;
      for (int sl = 0; sl < ns; ++sl) {
        int c = (int)(((run + c1 / 2) * (uint64_t)P) / (total ? total : 1));
        if (c >= P) c = P - 1;
        c = (c + rot) % P;
        std::vector<CtaPhase>& L = deal[s][c];
        if (!L.empty() && L.back().op == o && L.back().row0 + 16u * L.back().S == (uint32_t)sl * 16u) ++L.back().S;
        else L.push_back(CtaPhase{o, (uint32_t)sl * 16u, 1u});
        run += c1;
      }
    }
  }

  // 2. direct mode if every CTA can hold a stage's inputs whole
  const uint32_t kDirectCap = 40u * 1024u;
  bool direct = B <= 3;
  uint32_t xarea = 0;
  if (direct) {
    for (int s = 0; s < n_stages && direct; ++s)
      for (int c = 0; c < P && direct; ++c) {
        uint32_t need = 0;
        for (const CtaPhase& ph : deal[s][c]) {
          const rwkvq_desc& d = ops[ph.op].W_desc;
          need += (xrows_bytes(B, (uint32_t)d.ic_pad) + xsums_bytes((int)nbp, (uint32_t)d.ic_pad, d.method == RWKVQ_SQ) + 15u) & ~15u;
        }
        if (need > kDirectCap) direct = false;
        xarea = std::max(xarea, need);
      }
  }
  info->mode = direct ? MODE_DIRECT : MODE_PREPASS;

  // window geometry of the pre-pass mode: T tiles per window, the largest divisor of KT that fits
  const uint32_t kWinTarget = 18u * 1024u;
  auto tiles_per_window = [&](const rwkvq_desc& d) -> uint32_t {
    const uint32_t KT = (uint32_t)d.ic_pad / 256u;
    uint32_t best = 1;
    for (uint32_t T = 1; T <= KT; ++T) {
      if (KT % T) continue;
      const uint32_t need = xrows_bytes(B, T * 256u) + xsums_bytes((int)nbp, T * 256u, d.method == RWKVQ_SQ);
      if (need <= kWinTarget) best = T;
    }
    return best;
  };
  uint32_t xwin = 0;
  if (!direct) {
    for (int i = 0; i < n_ops; ++i) {
      const uint32_t T = tiles_per_window(ops[i].W_desc);
      const uint32_t need = xrows_bytes(B, T * 256u) + xsums_bytes((int)nbp, T * 256u, ops[i].W_desc.method == RWKVQ_SQ);
      xwin = std::max(xwin, (need + 127u) & ~127u);
    }
    info->nxb = 3; info->xwin_bytes = xwin;
    xarea = info->nxb * xwin;
  } else {
    info->nxb = 0; info->xwin_bytes = 0;
    xarea = (xarea + 127u) & ~127u;
  }

  // 3. shared-memory budget
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
  info->off_partial = info->off_hq + (uint32_t)CW * kHeaderRing * 64u;
  // Two sets of partial-sum slots where they are small, so that a CTA's second phase of a stage
  // starts without waiting for the first one's slices to be reduced.
  info->n_sets = direct ? 2u : 1u;
  info->off_x = (info->off_partial + info->n_sets * 2u * (uint32_t)CW * info->slot_floats * 4u + 127u) & ~127u;
  info->off_ring = info->off_x + xarea;
  if (!direct && info->off_ring + (uint32_t)CW * 2u * entry > kSmemLimit) {
    // two input windows instead of three leave room for a weight ring two records deep
    info->nxb = 2; xarea = info->nxb * xwin;
    info->off_ring = info->off_x + xarea;
  }
  if (info->off_ring + (uint32_t)CW * 2u * entry > kSmemLimit) return RWKVQ_EUNSUPPORTED;
  int depth = (int)((kSmemLimit - info->off_ring) / ((uint32_t)CW * entry));
  if (depth > kHeaderRing - 2) depth = kHeaderRing - 2;   // the header ring must reach past the copies in flight
  info->depth = depth;
  info->smem_bytes = info->off_ring + (uint32_t)CW * (uint32_t)depth * entry;

  // 4. pre-pass table and scratch: one region, reused by every stage (a stage's pre-pass starts only
  //    after the previous stage, and with it every copy out of the region, has finished everywhere)
  std::vector<StepMixOp> mixops(direct ? 0 : n_ops);
  std::vector<uint64_t> mix_x_off(n_ops, 0), mix_sums_off(n_ops, 0);
  uint64_t scratch_bytes = 0;
  if (!direct) {
    for (int s = 0; s < n_stages; ++s) {
      uint64_t off = 0;
      for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) {
        const rwkvq_gemv_op& op = ops[o];
        mix_x_off[o] = off; off += round_up_sz((size_t)B * op.W_desc.ic_pad * 2, 256);
        mix_sums_off[o] = off; off += round_up_sz((size_t)(op.W_desc.ic_pad / 128) * 3 * nbp * 4, 256);
        StepMixOp& m = mixops[o];
        std::memset(&m, 0, sizeof(m));
        m.x = (uint64_t)(uintptr_t)op.x_fp16_dev;
        if (op.mu_image_dev) {
          const uint8_t* mi = static_cast<const uint8_t*>(op.mu_image_dev);
          m.xprev = (uint64_t)(uintptr_t)op.xprev_fp16_dev;
          m.mu = (uint64_t)(uintptr_t)(mi + RWKVQ_HEADER_BYTES);
          m.mu_aux = (uint64_t)(uintptr_t)(mi + vector_aux_offset(&op.mu_desc));
          m.mu_bits = (uint16_t)op.mu_desc.bits; m.mu_entries = (uint16_t)op.mu_desc.entries;
        }
        m.dst_x = mix_x_off[o]; m.dst_sums = mix_sums_off[o];
        m.ic = (uint32_t)op.W_desc.ic; m.ic_pad = (uint32_t)op.W_desc.ic_pad;
        m.sums = op.W_desc.method == RWKVQ_SQ ? 1 : 0;
      }
      scratch_bytes = std::max(scratch_bytes, off);
    }
  }

  // 5. per-CTA descriptor lists
  std::vector<uint32_t> desc_off(P + 1, 0), init_post(P, 0);
  std::vector<PhaseDesc> descs;
  for (int c = 0; c < P; ++c) {
    desc_off[c] = (uint32_t)descs.size();
    uint32_t items = 0, win_seq = 0;
    // stages this CTA completes without consuming anything are reported with the previous stage
    // that has items (or at the start of the launch)
    std::vector<int> has_items(n_stages, 0);
    for (int s = 0; s < n_stages; ++s) has_items[s] = deal[s][c].empty() ? 0 : 1;
    int first_with = 0;
    while (first_with < n_stages && !has_items[first_with]) ++first_with;
    init_post[c] = (uint32_t)first_with;
    for (int s = 0; s < n_stages; ++s) {
      if (!direct) {
        PhaseDesc pd;
        std::memset(&pd, 0, sizeof(pd));
        pd.kind_flags = DK_PREPASS | DF_FIRST;
        pd.stage = (uint32_t)s;
        uint64_t G = 0;
        for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) G += (uint64_t)B * (ops[o].W_desc.ic_pad / 128);
        pd.S = (uint32_t)stage_ranges[s].first; pd.KT = (uint32_t)(stage_ranges[s].second - stage_ranges[s].first);
        pd.T = (uint32_t)(G * (uint64_t)c / P); pd.n_win = (uint32_t)(G * (uint64_t)(c + 1) / P);
        descs.push_back(pd);
      }
      if (!has_items[s]) continue;
      // sub-phases: in windowed mode a warp keeps at most two slices' accumulators, which needs S <= CW
      std::vector<CtaPhase> phases;
      for (const CtaPhase& ph : deal[s][c]) {
        const uint32_t T = direct ? (uint32_t)ops[ph.op].W_desc.ic_pad / 256u : tiles_per_window(ops[ph.op].W_desc);
        const bool windows = !direct && T < (uint32_t)ops[ph.op].W_desc.ic_pad / 256u;
        const uint32_t cap = windows ? (uint32_t)CW : (uint32_t)kCnt;   // and a phase's slices each own a counter
        for (uint32_t s0 = 0; s0 < ph.S; s0 += cap)
          phases.push_back(CtaPhase{ph.op, ph.row0 + 16u * s0, std::min<uint32_t>(cap, ph.S - s0)});
      }
      uint32_t stage_items = 0, n_slices = 0;
      for (const CtaPhase& ph : phases) { stage_items += ph.S * ((uint32_t)ops[ph.op].W_desc.ic_pad / 256u); n_slices += ph.S; }
      int next_with = s + 1;
      while (next_with < n_stages && !has_items[next_with]) ++next_with;
      uint32_t xo = 0, cnt = 0;
      for (size_t k = 0; k < phases.size(); ++k) {
        const CtaPhase& ph = phases[k];
        const rwkvq_gemv_op& op = ops[ph.op];
        const rwkvq_desc& d = op.W_desc;
        const uint8_t* img = static_cast<const uint8_t*>(op.W_image_dev);
        const bool sq = d.method == RWKVQ_SQ;
        PhaseDesc pd;
        std::memset(&pd, 0, sizeof(pd));
        // the slice counters are reused once the stage has gone through all of them: every warp
        // must then have left the phases that used them
        bool wrap = false;
        if (cnt + ph.S > (uint32_t)kCnt) { cnt = 0; wrap = true; }
        pd.kind_flags = DK_PHASE | ((uint32_t)fmt_of(d) << 4) | (k == 0 ? DF_FIRST : 0u) | (k + 1 == phases.size() ? DF_LAST : 0u) |
                        (op.mu_image_dev ? DF_MU : 0u) | (sq ? DF_SUMS : 0u) | ((k >= info->n_sets || wrap) ? DF_SYNC : 0u);
        pd.slot_set = (uint32_t)(k % info->n_sets);
        pd.stage = (uint32_t)s;
        pd.src = (uint64_t)(uintptr_t)(img + RWKVQ_HEADER_BYTES);
        pd.cb = sq ? 0 : (uint64_t)(uintptr_t)(img + matrix_aux_offset(&d));
        pd.y = (uint64_t)(uintptr_t)op.y_dev;
        pd.oc = (uint32_t)d.oc; pd.row0 = ph.row0; pd.S = ph.S; pd.KT = (uint32_t)d.ic_pad / 256u;
        pd.cnt_base = cnt; cnt += ph.S;
        pd.items_end = items + stage_items;
        pd.post_value = (uint32_t)next_with;
        pd.ic = (uint32_t)d.ic;
        if (direct) {
          pd.T = pd.KT; pd.n_win = 1;
          pd.xoff = xo; pd.xstride = (uint32_t)d.ic_pad * 2u + 32u;
          pd.gsoff = xo + xrows_bytes(B, (uint32_t)d.ic_pad);
          xo += (xrows_bytes(B, (uint32_t)d.ic_pad) + xsums_bytes((int)nbp, (uint32_t)d.ic_pad, sq) + 15u) & ~15u;
          pd.x = (uint64_t)(uintptr_t)op.x_fp16_dev;
          if (op.mu_image_dev) {
            const uint8_t* mi = static_cast<const uint8_t*>(op.mu_image_dev);
            pd.xprev = (uint64_t)(uintptr_t)op.xprev_fp16_dev;
            pd.mu = (uint64_t)(uintptr_t)(mi + RWKVQ_HEADER_BYTES);
            pd.mu_aux = (uint64_t)(uintptr_t)(mi + vector_aux_offset(&op.mu_desc));
            pd.mu_bits = (uint16_t)op.mu_desc.bits; pd.mu_entries = (uint16_t)op.mu_desc.entries;
          }
        } else {
          pd.T = tiles_per_window(d); pd.n_win = pd.KT / pd.T;
          pd.xoff = 0; pd.xstride = pd.T * 512u + 32u;
          pd.gsoff = xrows_bytes(B, pd.T * 256u);
          pd.win_seq0 = win_seq; win_seq += pd.n_win;
          pd.x = mix_x_off[ph.op]; pd.xprev = mix_sums_off[ph.op];
          pd.ic = (uint32_t)d.ic_pad * 2u;      // bytes between batch rows of x_mix in the scratch
        }
        descs.push_back(pd);
      }
      items += stage_items;
    }
    PhaseDesc end;
    std::memset(&end, 0, sizeof(end));
    end.kind_flags = DK_END;
    descs.push_back(end);
  }
  desc_off[P] = (uint32_t)descs.size();
  info->n_descs = (uint32_t)descs.size();

  size_t off = 256;
  info->off_desc_off = off; off += round_up_sz((size_t)(P + 1) * 4, 256);
  info->off_init_post = off; off += round_up_sz((size_t)P * 4, 256);
  info->off_descs = off; off += round_up_sz(descs.size() * sizeof(PhaseDesc), 256);
  info->off_flags = off; off += round_up_sz((size_t)P * 4, 256);
  info->off_flags2 = off; off += round_up_sz((size_t)P * 4, 256);
  info->off_mixops = off; off += round_up_sz(mixops.size() * sizeof(StepMixOp), 256);
  info->off_scratch = off; off += round_up_sz((size_t)scratch_bytes, 256);
  info->total_bytes = off;
  if (out) {
    out->assign(off, 0);
    memcpy(out->data() + info->off_desc_off, desc_off.data(), (size_t)(P + 1) * 4);
    memcpy(out->data() + info->off_init_post, init_post.data(), (size_t)P * 4);
    memcpy(out->data() + info->off_descs, descs.data(), descs.size() * sizeof(PhaseDesc));
    if (!mixops.empty()) memcpy(out->data() + info->off_mixops, mixops.data(), mixops.size() * sizeof(StepMixOp));
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
  info.abort_epoch = abort_epoch();   // the image just copied holds zeroed flags
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
    // needs no clearing pass.  A run that gave up leaves them uneven; start over after one.
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
  a.flags2 = reinterpret_cast<unsigned*>(pw + info.off_flags2);
  a.base = (info.runs - 1u) * (unsigned)info.n_stages;
  a.status = device_status_ptr();
  if (!a.status) return RWKVQ_ECUDA;
  a.poll_limit = info.poll_limit; a.wait_skew = info.wait_skew;
  a.B = info.B; a.nbp = (info.B + 1) & ~1; a.depth = info.depth;
  a.entry_bytes = info.entry_bytes; a.slot_floats = info.slot_floats;
  a.off_hq = info.off_hq; a.off_partial = info.off_partial; a.off_x = info.off_x; a.off_ring = info.off_ring;
  a.xwin_bytes = info.xwin_bytes; a.nxb = info.nxb;
  a.mixops = reinterpret_cast<const StepMixOp*>(p + info.off_mixops);
  a.scratch = pw + info.off_scratch;
  a.trace = static_cast<unsigned long long*>(info.trace_dev);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaSuccess;
  if (clear_flags) {
    e = cudaMemsetAsync(a.flags, 0, info.off_mixops - info.off_flags, s);
    if (e != cudaSuccess) return cuda_status(e);
  }
  const void* fn;
  if (info.trace_dev)
    fn = info.mode == MODE_DIRECT ? (const void*)step_kernel<1, MODE_DIRECT, kConsumerWarps, true>
         : info.NB == 1           ? (const void*)step_kernel<1, MODE_PREPASS, kConsumerWarps, true>
                                  : (const void*)step_kernel<2, MODE_PREPASS, kConsumerWarps, true>;
  else
    fn = info.mode == MODE_DIRECT ? (const void*)step_kernel<1, MODE_DIRECT, kConsumerWarps, false>
         : info.NB == 1           ? (const void*)step_kernel<1, MODE_PREPASS, kConsumerWarps, false>
                                  : (const void*)step_kernel<2, MODE_PREPASS, kConsumerWarps, false>;
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
  return (size_t)it->second.P * (size_t)(it->second.CW + 2) * kTraceSlots * sizeof(unsigned long long);
}

rwkvq_status rwkvq_step_trace(const void* plan_dev, void* trace_dev, size_t trace_bytes) {
  if (!plan_dev) return RWKVQ_EINVAL;
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  auto it = g_plans.find(plan_dev);
  if (it == g_plans.end()) return RWKVQ_EINVAL;
  if (trace_dev) {
    if (((uintptr_t)trace_dev & 7u) != 0) return RWKVQ_EALIGN;
    if (trace_bytes < (size_t)it->second.P * (size_t)(it->second.CW + 2) * kTraceSlots * sizeof(unsigned long long)) return RWKVQ_ENOMEM;
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
    for (uint32_t k = desc_off[c]; k < desc_off[c + 1]; ++k) {
      const PhaseDesc& d = descs[k];
      if ((d.kind_flags & 15u) != DK_PHASE) continue;
      auto it = op_of_y.find(d.y);
      if (it == op_of_y.end()) return RWKVQ_EINVAL;     // the walk needs distinct output buffers
      const int o = it->second;
      const uint32_t KT = d.KT, N = d.S * d.T;
      if (KT != (uint32_t)ops[o].W_desc.ic_pad / 256u || d.T * d.n_win != KT) return RWKVQ_EINVAL;
      // the walk of producer_role: every warp, every window, its share of the S x T grid
      for (uint32_t w = 0; w < (uint32_t)info.CW; ++w) {
        uint32_t i0, i1;
        item_range<kConsumerWarps>(N, w, i0, i1);
        for (uint32_t j = 0; j < d.n_win; ++j)
          for (uint32_t i = i0; i < i1; ++i) {
            const uint32_t sl = i / d.T, tt = i - sl * d.T;
            const uint32_t slice = d.row0 / 16u + sl, kt = j * d.T + tt;
            if (slice >= (uint32_t)ops[o].W_desc.oc / 16u || kt >= KT) return RWKVQ_EINVAL;
            counts_host[base[o] + (size_t)slice * KT + kt] += 1u;
            ++items;
          }
      }
      if (items > d.items_end) return RWKVQ_EINVAL;
      if ((d.kind_flags & DF_LAST) && items != d.items_end) return RWKVQ_EINVAL;
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
