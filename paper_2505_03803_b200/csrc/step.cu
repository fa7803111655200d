// A whole decode step as one persistent launch.
//
// Decode at batch 1..16 reads every packed weight once and does almost no arithmetic per byte
// (the paper's compute-to-memory argument, Section 1 and Appendix A.3), and one projection of a
// 7B-class layer is only a few microseconds of HBM time.  Launching one kernel per projection
// leaves the memory system idle between launches, so the step is ONE kernel with one CTA per SM:
//
//   * a producer warp streams packed weights from HBM into a ring of shared-memory slots with
//     bulk asynchronous copies (cp.async.bulk + mbarrier transaction counts).  Weights never depend
//     on activations, so the stream runs ahead across products and across stage boundaries;
//   * the stager warps (three, or seven for batches above 8: Shape) build the fp16 input x_mix = x + (x_prev - x) (.) mu_hat (Appendix A.1
//     Eq. 20) of the next run of units in one of two shared-memory buffers.  What does not depend
//     on the previous stage (mu_hat, x_prev) is prepared before the grid-wide stage barrier; the
//     stagers also clear the next stage's outputs and post this CTA's arrival at the barrier;
//   * consumer warps in groups of eight (two groups; one for batches above 8, whose record routine
//     needs the registers of two).  A unit is a 256-row x 256-column tile (two 128-row chunks of the
//     packed image); the groups take the CTA's units alternately, so one group computes while the
//     other waits, flushes or synchronises.  Warp w of a group owns rows
//     16w..16w+15 of both chunks and runs the m16n8k16 tensor-core steps of gemv_core.cuh with
//     every input fragment shared by the two records.  Partial sums go to y with fp32 reductions
//     (16 bytes per lane after a transpose among lanes) at the end of a run along K.
//
// For batches of four and more, and whenever a product's input is an element-wise operator on
// earlier outputs (rwkvq_input_xform: the WKV recurrence and sigmoid gate of Appendix A.1 Eqs. 23-24,
// the squared ReLU and output gate of Eq. 27, optionally a root-mean-square normalisation), the
// inputs of a stage are not built per CTA: after the stage barrier all CTAs together compute the
// stage's x_mix once (mix_slice: a half-warp per 128-column group) into a scratch region of the plan,
// publish it through a second barrier, and every CTA fetches its segments with bulk copies.
//
// The host plans the step once: every stage's units are dealt WHOLE to the CTAs, row of tiles by
// row of tiles where that balances (each row gets a number of CTAs by greedy cost per CTA), else at
// their cost midpoints, small stages in eighths of a unit (one warp's records); the plan is a per-CTA
// list of 128-byte unit descriptors plus a list of 64-byte input events (segments and barrier
// arrivals).
#include <cuda.h>           // types of the stream memory operations (no driver symbol is linked)
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
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

enum { UF_FLUSH = 1, UF_VQ = 2, UF_BITS8 = 4 };

struct StepUnit {            // 128 bytes, copied into the slot header by the producer
  uint64_t src0, src1;       // global addresses of the first copied record of chunk A / chunk B (0 = absent)
  uint64_t cb_src;           // VQ: codebook of the tile
  uint32_t bytes0, bytes1;   // bytes copied from each chunk: (w1 - w0) records
  uint32_t cb_bytes;
  uint32_t off0;             // w0 * record bytes: where the copied records sit inside a chunk
  uint32_t flags;            // UF_* | w0 << 8 | w1 << 12: warps w0 <= w < w1 of the group have a record
  uint32_t seg;              // number, within this CTA, of the input segment the unit reads
  uint32_t stage;            // stage number (0-based)
  uint32_t xcol0;            // column of the unit's tile inside the segment
  uint32_t row0, oc;         // first output row of chunk A; rows of the product
  uint64_t y;                // float y[B][oc]
  uint32_t xstride, gs_off;  // geometry of the segment: bytes between batch rows, offset of the sums
  uint32_t nbp, entries;
  uint32_t chunk_bytes;      // distance between chunk A and chunk B inside the slot
  uint32_t rec_bytes;
  uint32_t ev_index;         // position of the unit's segment in this CTA's event list
  uint32_t between_mask;     // events between the group's previous segment and this one, oldest in bit 0:
                             // 1 = barrier arrival, 0 = segment of the other group (valid for up to 32 events)
  uint32_t after_count;      // set on a group's last unit of a stage: events after its segment up to and
  uint32_t after_mask;       // including the stage's barrier arrival, to be passed right after the unit
  uint32_t pad[4];
};
static_assert(sizeof(StepUnit) == 128, "unit descriptor size");

enum { EV_SEGMENT = 0, EV_ARRIVE = 1 };

struct StepEvent {           // 64 bytes
  union {
    // segment.  Mixed in the CTA: x, xprev, mu, mu_aux as given by the caller.  Copied from the
    // stage's pre-pass (StepArgs::mix): x = first byte of the segment in the pre-pass rows,
    // xprev = first byte of its sums, mu = 0.
    struct { uint64_t x, xprev, mu, mu_aux; } seg;
    // arrival: float ranges to clear before arriving; then this CTA's share of the stage's
    // pre-pass: groups [grp_lo, grp_hi) of the stage's (product, batch row, 128-column group) list
    struct { uint64_t zptr[3]; uint32_t grp_lo, grp_hi; } arr;
  };
  union {
    struct { uint32_t ic, col0, ncols; uint16_t mu_bits, mu_entries; } segd;   // copied segments: ic = bytes between rows
    struct { uint32_t zcount[3]; uint16_t op_first, op_count; } arrd;          // products of the stage the pre-pass covers
  };
  uint32_t kind;             // EV_SEGMENT / EV_ARRIVE
  uint32_t barrier;          // segment: index + 1 of the stage barrier to pass first; arrival: index of the barrier
  uint32_t xstride_sums;     // segment: xstride | sums << 31
  uint16_t mu_off16;         // segment: offset / 16 of the decoded mu row inside the buffer
  uint16_t reserved;
};
static_assert(sizeof(StepEvent) == 64, "event descriptor size");

// One product's share of a stage's pre-pass: where its inputs are and where x_mix (fp16 rows of
// ic_pad columns, zero beyond ic) and the per-group sums ([group][3][nbp] floats) go.
struct StepMixOp {           // 64 bytes
  uint64_t x, xprev, mu, mu_aux, dst_x, dst_sums;
  uint32_t ic, ic_pad;
  // kind: rwkvq_input_kind | 0x100 when the row is RMS-normalised | 0x200 when this token's input is stored
  // (xprev_out) | 0x400 on the first product of a stage in which some input is normalised | 0x800 on the first
  // product of a stage whose inputs are all plain buffers; a kind with any of the low ten bits set has a
  // StepMixX beside it
  uint16_t mu_bits, mu_entries, sums, kind;
};
static_assert(sizeof(StepMixOp) == 64, "pre-pass descriptor size");
// Element-wise operator in front of the product (rwkvq_input_xform): fp32 sources [B][ic], state,
// parameters.  Kept apart so that the pre-pass of plain products reads 64 bytes per item as before.
struct StepMixX {            // 80 bytes
  uint64_t src, k, v, state_a, state_b, state_p, u, w;   // `k` holds the gate for RWKVQ_IN_F32
  uint64_t xprev_out, scale;         // scale: device address of one float that multiplies the operator's result (0 = none)
};
static_assert(sizeof(StepMixX) == 80, "pre-pass operator descriptor size");

constexpr int kGroupWarps = 8, kGroupThreads = kGroupWarps * 32;
// Thread layout of a CTA, by the number of batch blocks NB a record is multiplied with.
//   NB = 1 (B <= 8): two consumer groups of eight warps, three stager warps, one producer warp: 640 threads,
//     96 registers each at launch, re-divided at entry (consumers kConsumerRegs, the last warpgroup
//     kStagerRegs).
//   NB = 2 (B > 8): the record routine wants about 150 registers, which sixteen consumer warps cannot have,
//     and eight warps that keep everything in registers outrun sixteen that spill: ONE consumer group,
//     seven stager warps (the stage pre-pass is theirs), one producer: 512 threads, 128 registers at
//     launch, re-divided to 152 for the two consumer warpgroups (what their routine needs to keep
//     everything in registers) and 104 for the other two (measured: 168 / 88 and 144 / 112 are slower).
template <int NB> struct Shape {
  static constexpr int kGroups = NB == 2 ? 1 : 2;
  static constexpr int kStagerWarps = NB == 2 ? 7 : 3;
  static constexpr int kConsumerWarps = kGroupWarps * kGroups;
  static constexpr int kConsumerThreads = kConsumerWarps * 32, kStagerThreads = kStagerWarps * 32;
  static constexpr int kThreads = kConsumerThreads + kStagerThreads + 32;
  static constexpr int kLaunchRegs = NB == 2 ? 128 : 96;
  static constexpr int kConsumerRegs = NB == 2 ? 152 : 104, kStagerRegs = NB == 2 ? 104 : 64;
  static_assert(kConsumerWarps % 4 == 0 && (kStagerWarps + 1) % 4 == 0, "register re-division works on warpgroups of four warps");
  static_assert(kConsumerRegs * kConsumerThreads + kStagerRegs * (kStagerThreads + 32) <= kLaunchRegs * kThreads,
                "register re-division exceeds the launch's pool");
  static_assert(kLaunchRegs * kThreads <= 65536, "register file");
};
constexpr int groups_of(int NB) { return NB == 2 ? 1 : 2; }
constexpr int threads_of(int NB) { return NB == 2 ? Shape<2>::kThreads : Shape<1>::kThreads; }
constexpr int kMaxSlots = 12;
constexpr uint32_t kCtrlBytes = 1024, kXBufTotal = 65536, kMuScratch = 1024;
// Input-segment buffers: two of 32 KB, one in use and one being filled.  Large segments matter more than
// deep buffering (every hand-over of a segment costs all roles a pass through the barriers): four buffers
// of a quarter the size, and buffers that cost the weight ring a slot or two, were measured and are slower.
template <bool MIX, int NB> struct XBufs { static constexpr uint32_t kCount = 2u, kBytes = kXBufTotal / kCount; };
constexpr uint32_t kSmemLimit = 232448;  // 227 KB
constexpr uint32_t kDefaultPollLimit = 1u << 22;

struct StepArgs {
  const StepUnit* units;
  const StepEvent* events;
  const uint32_t* unit_off;   // [P+1]
  const uint32_t* event_off;  // [P+1]
  unsigned* counter;          // stage barriers: arrivals at barrier k, summed over all runs, in counter[k]
  unsigned target;            // arrivals that open a barrier in this run: run number * CTAs (mod 2^32)
  unsigned wait_skew;         // added to the target the WAITS compare with (0; a test sets it to make them run out)
  uint32_t poll_limit;        // polls after which a wait gives up
  int* status;
  int B, n_slots, n_stages;
  uint32_t slot_bytes, replica_bytes;
  // Larger batches: x_mix and the sums of a stage are computed ONCE by all CTAs together after the
  // stage barrier (instead of by every CTA that reads a column), published through a second
  // barrier per stage (counter[n_stages + 1 + s]), and fetched into the segment buffers with bulk copies.
  int mix;
  const StepMixOp* mixops;    // dst_x / dst_sums are offsets into `scratch`
  const StepMixX* mixx;       // parallel to mixops
  uint8_t* scratch;
  // Host-buffer runs (rwkvq_step_run_host): the activations arrive in chunks of 2^in_shift bytes while
  // the step is already running; after chunk i the copy stream stores in_base + i + 1 in *in_flag.
  // Whoever reads inputs inside [in_lo, in_hi) first waits for the chunk that holds their last byte.
  // in_flag == nullptr: the inputs are resident.
  const unsigned* in_flag;
  unsigned in_base, in_shift;
  uint64_t in_lo, in_hi;
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
// The launch's poll limit sits directly behind the CTA's abort flag in the control block (Ctrl).
__device__ __forceinline__ uint32_t poll_limit_of(volatile int* abort_flag) { return (uint32_t)abort_flag[1]; }
// Bounded wait by one thread: gives up (and raises the CTA-wide abort flag) after that many polls
// or when another role of this CTA has already given up.
__device__ __forceinline__ bool mbar_wait_one(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  const uint32_t limit = poll_limit_of(abort_flag);
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(status, (int)RWKVQ_ETIMEOUT);
  return false;
}
// Warp-collective bounded wait: every lane polls (so that each lane itself observes the completed
// phase and with it the data the barrier guards); the verdict is made warp-uniform.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  const bool ok = mbar_wait_one(bar, parity, abort_flag, status);
  return __all_sync(0xFFFFFFFFu, ok);
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
__device__ __forceinline__ void bulk_g2s_plain(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_sys(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_gpu(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t smem_add_acq_rel(uint32_t* p, uint32_t v) {
  uint32_t old;
  asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(smem_u32(p)), "r"(v) : "memory");
  return old;
}

struct Ctrl {
  uint64_t full[kMaxSlots], empty[kMaxSlots];
  uint64_t xfull[4], xempty[4];
  uint32_t stage_cnt[64];    // one 8-bit count per grid barrier (four per word): how many of the parties
                             // of this CTA (every consumer warp, and the stagers as one) have reported the
                             // stage that the barrier closes.  Per barrier, not one running total: consumer
                             // warps of a CTA without work in the coming stages may run any number of
                             // stages ahead of the stagers.
  int abort_flag;
  int poll_limit;            // must follow abort_flag (poll_limit_of)
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block");
constexpr uint32_t kMaxBarriers = 256;   // barriers that close a stage (8-bit counts in Ctrl::stage_cnt)

// One of the parties of grid barrier `b` (each consumer warp, the stagers as one) reports that its part of the stage the barrier
// closes is done; whoever reports last posts the CTA's arrival.  The count is an acquire-release
// read-modify-write at CTA scope and the arrival a GPU-scope release, so the arrival is ordered
// after everything every party did before reporting (the consumers' reductions into y, the
// stagers' clearing of the next outputs): block-level synchronisation followed by one thread's
// release, the pattern of a cooperative grid barrier.
template <int NB>
__device__ __forceinline__ void stage_report(Ctrl* ctrl, const StepArgs& a, uint32_t b) {
  const uint32_t sh = 8u * (b & 3u);
  const uint32_t old = smem_add_acq_rel(&ctrl->stage_cnt[b >> 2], 1u << sh);
  if (((old >> sh) & 0xFFu) == (uint32_t)Shape<NB>::kConsumerWarps) red_release_gpu(a.counter + b, 1u);
}
// Where the consumer warps are the busy role (two batch blocks per record) they only count
// themselves in, and a stager thread, which has nothing else to do at that point, waits (bounded)
// for the consumer warps' reports of THIS barrier and arrives: the release, which waits for the CTA's
// outstanding reductions, stays off the consumer warps.  The count is per barrier (the 8-bit
// fields of stage_cnt): a warp without work in the next stages runs ahead through their events,
// so a running total over all stages would reach its value for this stage while warps of
// this stage are still adding to the outputs.
__device__ __forceinline__ void stage_report_total(Ctrl* ctrl, uint32_t b) {
  asm volatile("red.release.cta.shared::cta.add.u32 [%0], %1;" ::"r"(smem_u32(&ctrl->stage_cnt[b >> 2])), "r"(1u << (8u * (b & 3u))) : "memory");
}
template <int NB>
__device__ __forceinline__ bool stage_wait_total_and_arrive(Ctrl* ctrl, const StepArgs& a, uint32_t b, volatile int* abort_flag) {
  const uint32_t limit = poll_limit_of(abort_flag) << 4;
  const uint32_t sh = 8u * (b & 3u);
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(&ctrl->stage_cnt[b >> 2])) : "memory");
    if (((v >> sh) & 0xFFu) >= (uint32_t)Shape<NB>::kConsumerWarps) { red_release_gpu(a.counter + b, 1u); return true; }
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(a.status, (int)RWKVQ_ETIMEOUT);
  return false;
}

// One thread: wait (bounded) until the chunk that holds byte `last` (the address of the last input byte
// about to be read) has arrived.  Addresses outside the arriving range are resident already.
__device__ __forceinline__ bool wait_inputs(const StepArgs& a, uint64_t last, volatile int* abort_flag) {
  if (!a.in_flag || last < a.in_lo || last >= a.in_hi) return true;
  const unsigned need = a.in_base + (unsigned)((last - a.in_lo) >> a.in_shift) + 1u;
  const uint32_t limit = a.poll_limit << 2;
  for (uint32_t it = 0; it < limit; ++it) {
    if ((int)(ld_acquire_sys(a.in_flag) - need) >= 0) return true;
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(a.status, (int)RWKVQ_ETIMEOUT);
  return false;
}

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
      // fields for lane 0, by 16-byte piece of descriptor k
      const uint32_t s0l = __shfl_sync(0xFFFFFFFFu, cur.x, 8 * k), s0h = __shfl_sync(0xFFFFFFFFu, cur.y, 8 * k);
      const uint32_t s1l = __shfl_sync(0xFFFFFFFFu, cur.z, 8 * k), s1h = __shfl_sync(0xFFFFFFFFu, cur.w, 8 * k);
      const uint32_t cbl = __shfl_sync(0xFFFFFFFFu, cur.x, 8 * k + 1), cbh = __shfl_sync(0xFFFFFFFFu, cur.y, 8 * k + 1);
      const uint32_t by0 = __shfl_sync(0xFFFFFFFFu, cur.z, 8 * k + 1), by1 = __shfl_sync(0xFFFFFFFFu, cur.w, 8 * k + 1);
      const uint32_t cbb = __shfl_sync(0xFFFFFFFFu, cur.x, 8 * k + 2), off0 = __shfl_sync(0xFFFFFFFFu, cur.y, 8 * k + 2);
      const uint32_t chb = __shfl_sync(0xFFFFFFFFu, cur.z, 8 * k + 5);
      __syncwarp();
      if (lane == 0) {
        const uint32_t tx = by0 + by1 + cbb;
        uint64_t* full = &ctrl->full[slot];
        if (tx == 0) {
          mbar_arrive(full);
        } else {
          mbar_arrive_expect_tx(full, tx);
          uint8_t* data = sl + 128;
          if (by0) bulk_g2s(data + off0, reinterpret_cast<const void*>(((uint64_t)s0h << 32) | s0l), by0, full, policy);
          if (by1) bulk_g2s(data + chb + off0, reinterpret_cast<const void*>(((uint64_t)s1h << 32) | s1l), by1, full, policy);
          if (cbb) bulk_g2s(data + 2 * chb, reinterpret_cast<const void*>(((uint64_t)cbh << 32) | cbl), cbb, full, policy);
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
      for (uint32_t it = 0; it < a.poll_limit; ++it)
        if (mbar_try_wait(&ctrl->full[slot], parity)) break;
    }
  }
}

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

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + expf(-x)); }
__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// Eight consecutive inputs of a product from the element-wise operator in front of it (Appendix A.1
// Eqs. 23, 24, 27), rounded to fp16.  e0: index of the first element in the [B][ic] fp32 arrays,
// col: its column (index into the per-channel parameters).  `commit` false (a lane that repeats
// another lane's group to keep the half-warp whole): the recurrence state is not written.
__device__ __forceinline__ uint4 xform_input(const StepMixOp& mo, const StepMixX& op, size_t e0, int col, bool commit, float rstd) {
  float s[8];
  {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(op.src) + e0));
    const float4 c = __ldcg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(op.src) + e0 + 4));
    s[0] = a.x; s[1] = a.y; s[2] = a.z; s[3] = a.w; s[4] = c.x; s[5] = c.y; s[6] = c.z; s[7] = c.w;
  }
  float o[8];
  const int kind = mo.kind & 0xFF;
  if (kind == RWKVQ_IN_RELU2) {
#pragma unroll
    for (int i = 0; i < 8; ++i) { const float m = fmaxf(s[i], 0.f); o[i] = m * m; }
  } else if (kind == RWKVQ_IN_F32) {
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = s[i];
    if (op.k) {      // gate
      const float* g = reinterpret_cast<const float*>(op.k) + e0;
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] *= sigmoidf_(__ldcg(g + i));
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] *= rstd;
  } else {           // RWKVQ_IN_WKV
    const float* kp = reinterpret_cast<const float*>(op.k) + e0;
    const float* vp = reinterpret_cast<const float*>(op.v) + e0;
    float* sa = reinterpret_cast<float*>(op.state_a) + e0;
    float* sb = reinterpret_cast<float*>(op.state_b) + e0;
    float* sp = reinterpret_cast<float*>(op.state_p) + e0;
    const float* up = reinterpret_cast<const float*>(op.u) + col;
    const float* wp = reinterpret_cast<const float*>(op.w) + col;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      // the history sums are stored as a = e^{-p} sum f v, b = e^{-p} sum f; every exponential below has
      // a non-positive argument
      const float k = __ldcg(kp + i), vv = __ldcg(vp + i), a = __ldcg(sa + i), bb = __ldcg(sb + i), p = __ldcg(sp + i);
      const float uk = __ldg(up + i) + k;
      const float q = fmaxf(p, uk);
      const float e1 = expf(p - q), e2 = expf(uk - q);
      const float wkv = (e1 * a + e2 * vv) / (e1 * bb + e2);
      o[i] = sigmoidf_(s[i]) * wkv;
      const float pw = p - __ldg(wp + i);
      const float q2 = fmaxf(pw, k);
      const float f1 = expf(pw - q2), f2 = expf(k - q2);
      if (commit) { sa[i] = f1 * a + f2 * vv; sb[i] = f1 * bb + f2; sp[i] = q2; }
    }
  }
  if (op.scale) {
    const float gsc = __ldcg(reinterpret_cast<const float*>(op.scale));
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] *= gsc;
  }
  return make_uint4(pack_half2(o[0], o[1]), pack_half2(o[2], o[3]), pack_half2(o[4], o[5]), pack_half2(o[6], o[7]));
}

// 1 / sqrt(mean over the row of v^2 + 1e-6), v = src (* sigmoid(gate)): the sixteen lanes of a half-warp
// read row b of the fp32 source(s) together.  Items that follow one another in a half-warp mostly share
// the row, so the caller keeps the last result.
// Called by whole warps (the shuffles name all 32 lanes); a half-warp with `active` false reads nothing.
__device__ __forceinline__ float row_rstd(const StepMixOp& op, const StepMixX& ox, int b, int l16, bool active) {
  const float* src = reinterpret_cast<const float*>(ox.src) + (size_t)b * op.ic;
  const float* gate = ox.k ? reinterpret_cast<const float*>(ox.k) + (size_t)b * op.ic : nullptr;
  float acc = 0.f;
  for (uint32_t c = (uint32_t)l16 * 4u; active && c < op.ic; c += 64u) {
    float4 v = __ldcg(reinterpret_cast<const float4*>(src + c));
    if (gate) {
      const float4 g = __ldcg(reinterpret_cast<const float4*>(gate + c));
      v.x *= sigmoidf_(g.x); v.y *= sigmoidf_(g.y); v.z *= sigmoidf_(g.z); v.w *= sigmoidf_(g.w);
    }
    acc += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  __syncwarp();
#pragma unroll
  for (int d = 8; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
  return rsqrtf(acc / (float)op.ic + 1e-6f);
}

// A load whose value is not needed: it brings the sector into this SM's L1.
__device__ __forceinline__ void touch_global(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(reinterpret_cast<uintptr_t>(p) & ~static_cast<uintptr_t>(3)));
}

// Asks for the line to be brought into L2 (the point of coherence: a later write by another CTA, reduction
// or plain store, is seen by the load that follows).
__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" :: "l"(p));
}

// A pre-pass descriptor through the read-only path, so that the copy read ahead by mix_warm is found in L1.
__device__ __forceinline__ StepMixOp load_mixop(const StepMixOp* p) {
  union { StepMixOp op; uint4 q[4]; } u;
#pragma unroll
  for (int i = 0; i < 4; ++i) u.q[i] = __ldg(reinterpret_cast<const uint4*>(p) + i);
  return u.op;
}

// Everything mix_slice will read that does not depend on the stage before -- the products' descriptors,
// the mu_hat codes of this CTA's items and the codebook entries they select -- is read once ahead of
// time, while the consumer warps are still busy with the current stage, so that behind the barrier the
// chain of dependent loads (descriptor -> codes -> codebook) hits in L1 and only x itself comes from L2.
template <int NB>
__device__ void mix_warm(const StepArgs& a, const StepEvent& ev, int stid) {
  constexpr int kStagerWarps = Shape<NB>::kStagerWarps;
  const int lane = stid & 31, l16 = lane & 15;
  const uint32_t lo = ev.arr.grp_lo, hi = ev.arr.grp_hi;
  const StepMixOp* ops = a.mixops + ev.arrd.op_first;
  const int n_ops = (int)ev.arrd.op_count;
  if (lo >= hi) return;
  touch_global(reinterpret_cast<const uint8_t*>(ops) + 32);
  for (uint32_t g0 = lo + 2u * (uint32_t)(stid >> 5); g0 < hi; g0 += 2u * (uint32_t)kStagerWarps) {
    const uint32_t gi = g0 + (uint32_t)(lane >> 4);
    uint32_t r = gi < hi ? gi : lo;
    int k = 0;
    uint32_t icp = __ldg(&ops[0].ic_pad);
    while (k + 1 < n_ops && r >= (uint32_t)a.B * (icp >> 7)) { r -= (uint32_t)a.B * (icp >> 7); ++k; icp = __ldg(&ops[k].ic_pad); }
    const StepMixOp* op = ops + k;
    touch_global(op);                                            // both 32-byte sectors of the descriptor
    touch_global(reinterpret_cast<const uint8_t*>(op) + 32);
    const uint64_t mu = __ldg(&op->mu);
    const uint32_t kind = __ldg(&op->kind);
    if (kind) {
      const uint8_t* ox = reinterpret_cast<const uint8_t*>(a.mixx + ev.arrd.op_first + k);
      touch_global(ox); touch_global(ox + 32); touch_global(ox + 64); touch_global(ox + 76);
    }
    const uint32_t ic = __ldg(&op->ic);
    const uint32_t ng = icp >> 7;
    const int col = (int)(r % ng) * 128 + l16 * 8;
    // Inputs that no earlier stage of this step writes (the first products' x, every x_prev) are still in
    // HBM: ask for them now.  Inputs an earlier stage writes are in L2 already and the request is void.
    if ((kind & 0xFFu) == RWKVQ_IN_BUFFER && col < (int)ic && (l16 & 1) == 0) {
      const size_t e0 = (size_t)(r / ng) * ic + col;
      prefetch_l2(reinterpret_cast<const __half*>(__ldg(&op->x)) + e0);
      if (mu) prefetch_l2(reinterpret_cast<const __half*>(__ldg(&op->xprev)) + e0);
    }
    if (mu && col < (int)ic) {
      const uint32_t bits = __ldg(&op->mu_bits), mask = (1u << bits) - 1u;
      const uint32_t byte = (uint32_t)(col >> 1) * bits >> 3;
      const uint32_t* w = reinterpret_cast<const uint32_t*>(mu) + (byte >> 2);
      const uint32_t sh = (byte & 3u) * 8u;
      const uint32_t wlo = __ldg(w);
      const uint32_t whi = (sh + 4u * bits > 32u) ? __ldg(w + 1) : 0u;
      const uint32_t f = __funnelshift_r(wlo, whi, sh);
      const uint32_t* cb = reinterpret_cast<const uint32_t*>(__ldg(&op->mu_aux));
      touch_global(cb + (f & mask));
      touch_global(cb + ((f >> bits) & mask));
      touch_global(cb + ((f >> (2 * bits)) & mask));
      touch_global(cb + ((f >> (3 * bits)) & mask));
    }
  }
}

// This CTA's share of a stage's pre-pass.  A half-warp takes one (product, batch row, 128-column
// group) at a time: it loads x (and x_prev, and decodes mu_hat), mixes, rounds to fp16, stores the
// 128 values to the product's pre-pass rows and reduces the three sums of the group with shuffles.
template <int NB>
__device__ void mix_slice(const StepArgs& a, const StepEvent& ev, int stid) {
  constexpr int kStagerWarps = Shape<NB>::kStagerWarps, kStagerThreads = Shape<NB>::kStagerThreads;
  const int lane = stid & 31, l16 = lane & 15;
  const uint32_t lo = ev.arr.grp_lo, hi = ev.arr.grp_hi;
  const StepMixOp* ops = a.mixops + ev.arrd.op_first;
  const int n_ops = (int)ev.arrd.op_count;
  const int nbp = (a.B + 1) & ~1;
  // Row statistics first: the rows of normalised inputs that this CTA's items fall in (a few: the items
  // are consecutive groups of consecutive rows) are reduced by all stager threads together, 1.5 KB per
  // round of loads, into a small table; rows beyond the table are reduced by the half-warp that meets them.
  constexpr int kRowTable = 8;
  __shared__ float s_rstd[kRowTable];
  __shared__ float s_part[kStagerWarps];
  __shared__ uint32_t s_row_end[kRowTable];      // first item behind the row of each entry
  int n_rows = 0;
  const uint32_t stage_kind = __ldg(&ops[0].kind);
  if (stage_kind & 0x800) {
    // Stage of plain inputs (no operator, no normalisation): a quarter-warp per item, sixteen columns per
    // lane, so that a CTA's share is done in one round of loads.
    const int l8 = lane & 7;
    for (uint32_t g0 = lo + 4u * (uint32_t)(stid >> 5); g0 < hi; g0 += 4u * (uint32_t)kStagerWarps) {
      const uint32_t gi = g0 + (uint32_t)(lane >> 3);
      const bool valid = gi < hi;
      uint32_t r = valid ? gi : lo;
      int k = 0;
      uint32_t icp = __ldg(&ops[0].ic_pad);
      while (k + 1 < n_ops && r >= (uint32_t)a.B * (icp >> 7)) { r -= (uint32_t)a.B * (icp >> 7); ++k; icp = __ldg(&ops[k].ic_pad); }
      const StepMixOp op = load_mixop(ops + k);
      const uint32_t ng = op.ic_pad >> 7;
      const int b = (int)(r / ng), grp = (int)(r % ng);
      const int col = grp * 128 + l8 * 16;
      const size_t e0 = (size_t)b * op.ic + col;
      const bool in0 = col < (int)op.ic, in1 = col + 8 < (int)op.ic;
      uint4 v[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
      uint4 pr[2] = {v[0], v[0]};
      uint32_t f[2] = {0u, 0u};
      const __half* xs = reinterpret_cast<const __half*>(op.x) + e0;
      if (in0) v[0] = __ldcg(reinterpret_cast<const uint4*>(xs));
      if (in1) v[1] = __ldcg(reinterpret_cast<const uint4*>(xs + 8));
      if (op.mu) {
        const __half* ps = reinterpret_cast<const __half*>(op.xprev) + e0;
        if (in0) pr[0] = __ldcg(reinterpret_cast<const uint4*>(ps));
        if (in1) pr[1] = __ldcg(reinterpret_cast<const uint4*>(ps + 8));
        const uint32_t bits = op.mu_bits;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h == 0 ? in0 : in1) {
            // four indices = 4*bits bits starting at a byte boundary (col/2 is a multiple of 4)
            const uint32_t byte = (uint32_t)((col + 8 * h) >> 1) * bits >> 3;
            const uint32_t* w = reinterpret_cast<const uint32_t*>(op.mu) + (byte >> 2);
            const uint32_t sh = (byte & 3u) * 8u;
            const uint32_t wlo = __ldg(w);
            const uint32_t whi = (sh + 4u * bits > 32u) ? __ldg(w + 1) : 0u;
            f[h] = __funnelshift_r(wlo, whi, sh);
          }
        }
        const uint32_t mask = (1u << bits) - 1u;
        const uint32_t* cb = reinterpret_cast<const uint32_t*>(op.mu_aux);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (h == 0 ? in0 : in1) {
            v[h].x = mix2(v[h].x, pr[h].x, __ldg(cb + (f[h] & mask)));
            v[h].y = mix2(v[h].y, pr[h].y, __ldg(cb + ((f[h] >> bits) & mask)));
            v[h].z = mix2(v[h].z, pr[h].z, __ldg(cb + ((f[h] >> (2 * bits)) & mask)));
            v[h].w = mix2(v[h].w, pr[h].w, __ldg(cb + ((f[h] >> (3 * bits)) & mask)));
          }
        }
      }
      if (valid) {
        __half* dst = reinterpret_cast<__half*>(a.scratch + op.dst_x) + (size_t)b * op.ic_pad + col;
        *reinterpret_cast<uint4*>(dst) = v[0];
        *reinterpret_cast<uint4*>(dst + 8) = v[1];
      }
      // both vectors of a lane lie in one 16-column span of a triple: the same two bias values
      const int o = (16 * l8) & 63;
      const float pa = pair_sum(v[0].x) + pair_sum(v[0].z) + pair_sum(v[1].x) + pair_sum(v[1].z);
      const float pb = pair_sum(v[0].y) + pair_sum(v[0].w) + pair_sum(v[1].y) + pair_sum(v[1].w);
      float sx = pa + pb;
      float t0 = fmaf((float)rwkvq_sq_bias(o, 0), pa, (float)rwkvq_sq_bias(o + 2, 0) * pb);
      float t1 = fmaf((float)rwkvq_sq_bias(o, 1), pa, (float)rwkvq_sq_bias(o + 2, 1) * pb);
#pragma unroll
      for (int d = 4; d > 0; d >>= 1) {
        sx += __shfl_xor_sync(0xFFFFFFFFu, sx, d);
        t0 += __shfl_xor_sync(0xFFFFFFFFu, t0, d);
        t1 += __shfl_xor_sync(0xFFFFFFFFu, t1, d);
      }
      if (valid && l8 == 0 && op.sums) {
        float* gs = reinterpret_cast<float*>(a.scratch + op.dst_sums);
        gs[(grp * 3 + 0) * nbp + b] = sx;
        gs[(grp * 3 + 1) * nbp + b] = t0;
        gs[(grp * 3 + 2) * nbp + b] = t1;
      }
    }
    return;
  }
  if (stage_kind & 0x400) {      // the planner marks the first product of a stage that has a normalised input
    uint32_t r = lo;
    while (r < hi && n_rows < kRowTable) {
      uint32_t rr = r;
      int k = 0;
      uint32_t icp = __ldg(&ops[0].ic_pad);
      while (k + 1 < n_ops && rr >= (uint32_t)a.B * (icp >> 7)) { rr -= (uint32_t)a.B * (icp >> 7); ++k; icp = __ldg(&ops[k].ic_pad); }
      const StepMixOp op = ops[k];
      const uint32_t ng = op.ic_pad >> 7;
      const int b = (int)(rr / ng);
      float rstd = 1.f;
      if (op.kind & 0x100) {
        const StepMixX ox = a.mixx[ev.arrd.op_first + k];
        const float* src = reinterpret_cast<const float*>(ox.src) + (size_t)b * op.ic;
        const float* gate = ox.k ? reinterpret_cast<const float*>(ox.k) + (size_t)b * op.ic : nullptr;
        float acc = 0.f;
#pragma unroll 4
        for (uint32_t c = (uint32_t)stid * 4u; c < op.ic; c += (uint32_t)kStagerThreads * 4u) {
          float4 v = __ldcg(reinterpret_cast<const float4*>(src + c));
          if (gate) {
            const float4 g = __ldcg(reinterpret_cast<const float4*>(gate + c));
            v.x *= sigmoidf_(g.x); v.y *= sigmoidf_(g.y); v.z *= sigmoidf_(g.z); v.w *= sigmoidf_(g.w);
          }
          acc += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
        if (lane == 0) s_part[stid >> 5] = acc;
        named_bar_sync(5, kStagerThreads);
        float tot = 0.f;
#pragma unroll
        for (int wdx = 0; wdx < kStagerWarps; ++wdx) tot += s_part[wdx];
        rstd = rsqrtf(tot / (float)op.ic + 1e-6f);
        named_bar_sync(5, kStagerThreads);      // s_part is reused by the next row
      }
      r += ng - rr % ng;                         // first item of the next row
      if (stid == 0) { s_rstd[n_rows] = rstd; s_row_end[n_rows] = r; }
      ++n_rows;
    }
    named_bar_sync(5, kStagerThreads);
  }
  uint64_t stat_src = 0;     // row whose statistic this half-warp computed last (rows beyond the table)
  int stat_b = -1;
  float stat_rstd = 1.f;
  for (uint32_t g0 = lo + 2u * (uint32_t)(stid >> 5); g0 < hi; g0 += 2u * (uint32_t)kStagerWarps) {
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
    StepMixX ox;
    if (op.kind) ox = a.mixx[ev.arrd.op_first + k];
    else { ox.src = ox.k = ox.xprev_out = ox.scale = 0; }
    float rstd = 1.f;
    if (op.kind & 0x100) {
      // the two half-warps of a warp hold different items: the statistic is computed by the whole warp
      // whenever either half needs a new one
      const bool norm = (op.kind & 0x100) != 0;
      const uint32_t item = valid ? gi : lo;
      int idx = 0;
      while (idx < n_rows && item >= s_row_end[idx]) ++idx;
      const bool tabled = idx < n_rows;
      const bool want = norm && !tabled && (stat_src != ox.src || stat_b != b);
      if (__any_sync(0xFFFFFFFFu, want)) {
        const float rs = row_rstd(op, ox, b, l16, want);
        if (want) { stat_rstd = rs; stat_src = ox.src; stat_b = b; }
      }
      if (norm) rstd = tabled ? s_rstd[idx] : stat_rstd;
    }
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (col < (int)op.ic) {
      const size_t e0 = (size_t)b * op.ic + col;          // first of this lane's eight elements
      if ((op.kind & 0xFF) == RWKVQ_IN_BUFFER) v = __ldcg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(op.x) + e0));
      else v = xform_input(op, ox, e0, col, valid, rstd);
      if (ox.xprev_out || op.mu) {
        // previous token's input: read for the mix, then (where asked) replaced by this token's
        uint4 pr = make_uint4(0u, 0u, 0u, 0u);
        if (op.mu) pr = __ldcg(reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(op.xprev) + e0));
        if (ox.xprev_out && valid) *reinterpret_cast<uint4*>(reinterpret_cast<__half*>(ox.xprev_out) + e0) = v;
        if (op.mu) {
          const uint32_t bits = op.mu_bits, mask = (1u << bits) - 1u;
          // four indices = 4*bits bits starting at a byte boundary (col/2 is a multiple of 4)
          const uint32_t byte = (uint32_t)(col >> 1) * bits >> 3;
          const uint32_t* w = reinterpret_cast<const uint32_t*>(op.mu) + (byte >> 2);
          const uint32_t sh = (byte & 3u) * 8u;
          const uint32_t wlo = __ldg(w);
          const uint32_t whi = (sh + 4u * bits > 32u) ? __ldg(w + 1) : 0u;
          const uint32_t f = __funnelshift_r(wlo, whi, sh);
          const uint32_t* cb = reinterpret_cast<const uint32_t*>(op.mu_aux);
          v.x = mix2(v.x, pr.x, __ldg(cb + (f & mask)));
          v.y = mix2(v.y, pr.y, __ldg(cb + ((f >> bits) & mask)));
          v.z = mix2(v.z, pr.z, __ldg(cb + ((f >> (2 * bits)) & mask)));
          v.w = mix2(v.w, pr.w, __ldg(cb + ((f >> (3 * bits)) & mask)));
        }
      }
    }
    if (valid) *reinterpret_cast<uint4*>(reinterpret_cast<__half*>(a.scratch + op.dst_x) + (size_t)b * op.ic_pad + col) = v;
    const int o = (8 * l16) & 63;
    const float pa = pair_sum(v.x) + pair_sum(v.z), pb = pair_sum(v.y) + pair_sum(v.w);
    float sx = pa + pb;
    float t0 = fmaf((float)rwkvq_sq_bias(o, 0), pa, (float)rwkvq_sq_bias(o + 2, 0) * pb);
    float t1 = fmaf((float)rwkvq_sq_bias(o, 1), pa, (float)rwkvq_sq_bias(o + 2, 1) * pb);
#pragma unroll
    for (int d = 8; d > 0; d >>= 1) {
      sx += __shfl_xor_sync(0xFFFFFFFFu, sx, d);
      t0 += __shfl_xor_sync(0xFFFFFFFFu, t0, d);
      t1 += __shfl_xor_sync(0xFFFFFFFFu, t1, d);
    }
    if (valid && l16 == 0 && op.sums) {
      float* gs = reinterpret_cast<float*>(a.scratch + op.dst_sums);
      gs[(grp * 3 + 0) * nbp + b] = sx;
      gs[(grp * 3 + 1) * nbp + b] = t0;
      gs[(grp * 3 + 2) * nbp + b] = t1;
    }
  }
}

// Stagers walk the CTA's event list.
//  EV_ARRIVE: clear this CTA's slice of the next stage's outputs, then report the stage as done on
//    the stagers' side (stage_report: the last of the consumer warps and the stagers to report
//    adds this CTA's arrival to the grid barrier, so the arrival never waits for a role that is
//    busy with something else).
//  EV_SEGMENT: x_mix and, for SQ, the per-group sums of the segment, into buffer (segment number
//    & 1).  The decoded token-shift vector mu_hat and the previous token's activations go to
//    shared memory BEFORE the stage barrier, so that only one round of vector loads of x, the
//    mix and the sums remain behind it.  A thread owns 8 consecutive columns (16 bytes) of one
//    batch row; a half-warp owns one 128-column group, whose three sums it reduces with shuffles.
template <bool MIX, int NB>
__device__ void stager_role(const StepArgs& a, uint8_t* smem, Ctrl* ctrl, uint8_t* xbufs, uint32_t* mucb,
                            uint32_t e0, uint32_t e1) {
  constexpr int kStagerThreads = Shape<NB>::kStagerThreads;
  const int stid = threadIdx.x - Shape<NB>::kConsumerThreads;
  const int lane = stid & 31;
  volatile int* abortp = &ctrl->abort_flag;
  uint32_t nseg = 0;          // segments staged so far
  uint32_t passed2 = 0xFFFFFFFFu;   // second-stage barrier this CTA has already passed
  bool ok = true;
  for (uint32_t ei = e0; ei < e1; ++ei) {
    const StepEvent ev = *reinterpret_cast<const StepEvent*>(reinterpret_cast<const uint8_t*>(a.events) + (size_t)ei * 64);
    if (ev.kind == EV_ARRIVE) {
      if constexpr (MIX) {
        if (ev.barrier < (uint32_t)a.n_stages) mix_warm<NB>(a, ev, stid);
      }
#pragma unroll
      for (int k = 0; k < 3; ++k) {
        float* z = reinterpret_cast<float*>(ev.arr.zptr[k]);
        for (uint32_t e = stid; e < ev.arrd.zcount[k]; e += kStagerThreads) z[e] = 0.f;
      }
      // the clearing stores of every stager thread must precede thread 0's fence
      ok = named_bar_and(4, kStagerThreads, ok);
      if (!ok) break;
      // The stagers' part of the stage is done.  Barrier 0 (the clearing pass) has no consumer work
      // before it: arrive directly.  Otherwise report; the last party to report arrives.
      if (stid == 0) {
        if (ev.barrier == 0u) red_release_gpu(a.counter, 1u);
        else if constexpr (NB == 2) ok = stage_wait_total_and_arrive<NB>(ctrl, a, ev.barrier, abortp);
        else stage_report<NB>(ctrl, a, ev.barrier);
      }
      if constexpr (MIX) {
        // once the barrier opens, do this CTA's share of the new stage's pre-pass and publish it
        // through the stage's second barrier
        if (ev.barrier < (uint32_t)a.n_stages) {
          if (ok && stid == 0) {
            uint32_t it = 0;
            while ((int)(ld_acquire_gpu(a.counter + ev.barrier) - (a.target + a.wait_skew)) < 0) {
              if (++it >= (a.poll_limit << 2) || *abortp) { *abortp = 1; atomicExch(a.status, (int)RWKVQ_ETIMEOUT); ok = false; break; }
            }
            if (ok && a.in_flag) {
              // the last input byte any product of the coming stage reads (x and x_prev, [B][ic] fp16 each)
              const StepMixOp* mo = a.mixops + ev.arrd.op_first;
              uint64_t last = 0;
              for (uint32_t k = 0; k < ev.arrd.op_count; ++k) {
                const uint64_t span = (uint64_t)a.B * __ldg(&mo[k].ic) * 2u - 1u;
                const uint64_t px = __ldg(&mo[k].x), pp = __ldg(&mo[k].xprev);
                if (px >= a.in_lo && px < a.in_hi) last = max(last, px + span);
                if (pp >= a.in_lo && pp < a.in_hi) last = max(last, pp + span);
              }
              if (last) ok = wait_inputs(a, last, abortp);
            }
          }
          ok = named_bar_and(6, kStagerThreads, ok);   // thread 0's acquire precedes every thread's loads of x
          if (!ok) break;
          mix_slice<NB>(a, ev, stid);
          named_bar_sync(4, kStagerThreads);           // every thread's pre-pass stores precede thread 0's release
          if (stid == 0) red_release_gpu(a.counter + (uint32_t)a.n_stages + 1u + ev.barrier, 1u);
        }
      }
      continue;
    }
    const int buf = (int)(nseg % XBufs<MIX, NB>::kCount);
    // uniform verdict over all stager threads: the named barriers below must be reached by all or none
    ok = named_bar_and(7, kStagerThreads, mbar_wait_warp(&ctrl->xempty[buf], ((nseg / XBufs<MIX, NB>::kCount) & 1u) ^ 1u, abortp, a.status) && ok);
    uint8_t* xb = xbufs + (size_t)buf * XBufs<MIX, NB>::kBytes;
    if constexpr (MIX) {
      // The segment is a rectangle of the stage's pre-pass output: pass the stage's second barrier
      // (once per stage), then fetch B rows and the block of sums with bulk copies.
      const uint32_t b2 = (uint32_t)a.n_stages + ev.barrier;      // counter of the second barrier of stage ev.barrier - 1
      if (ok && stid == 0 && b2 != passed2) {
        uint32_t it = 0;
        while ((int)(ld_acquire_gpu(a.counter + b2) - (a.target + a.wait_skew)) < 0) {
          if (++it >= (a.poll_limit << 2) || *abortp) { *abortp = 1; atomicExch(a.status, (int)RWKVQ_ETIMEOUT); ok = false; break; }
        }
      }
      passed2 = b2;
      ok = named_bar_and(6, kStagerThreads, ok);
      if (ok && stid < 32) {
        const uint32_t xstride = ev.xstride_sums & 0x7FFFFFFFu;
        const uint32_t row_bytes = ev.segd.ncols * 2u;
        const uint32_t sums_bytes = (ev.xstride_sums >> 31) ? (ev.segd.ncols >> 7) * 3u * (uint32_t)((a.B + 1) & ~1) * 4u : 0u;
        // what other CTAs wrote with ordinary stores is read below by the copy engine
        asm volatile("fence.proxy.async;" ::: "memory");
        if (lane == 0) mbar_arrive_expect_tx(&ctrl->xfull[buf], (uint32_t)a.B * row_bytes + sums_bytes);
        __syncwarp();
        if (lane < a.B)
          bulk_g2s_plain(xb + (size_t)lane * xstride, a.scratch + ev.seg.x + (size_t)lane * ev.segd.ic, row_bytes, &ctrl->xfull[buf]);
        else if (lane == a.B && sums_bytes)
          bulk_g2s_plain(xb + (size_t)a.B * xstride, a.scratch + ev.seg.xprev, sums_bytes, &ctrl->xfull[buf]);
      } else if (lane == 0) {
        mbar_arrive(&ctrl->xfull[buf]);      // the other stager warps (and everyone after a failure) only arrive
      }
      ++nseg;
      if (!ok) break;
      continue;
    }
    const uint8_t* mu = reinterpret_cast<const uint8_t*>(ev.seg.mu);
    const __half* x = reinterpret_cast<const __half*>(ev.seg.x);
    const __half* xp = reinterpret_cast<const __half*>(ev.seg.xprev);
    const int ic = (int)ev.segd.ic, col0 = (int)ev.segd.col0;
    const uint32_t xstride = ev.xstride_sums & 0x7FFFFFFFu;
    const bool sums = (ev.xstride_sums >> 31) != 0;
    const int nvr = (int)ev.segd.ncols >> 3;            // 16-byte vectors per batch row
    const int total = a.B * nvr;
    const int nbp = (a.B + 1) & ~1;
    uint8_t* murow = xb + (size_t)ev.mu_off16 * 16;
    if (a.in_flag) {      // uniform: host-buffer run
      if (ok && stid == 0) {
        const uint64_t span = ((uint64_t)(a.B - 1) * (uint64_t)ic + (uint64_t)min(ic, col0 + (int)ev.segd.ncols)) * 2u - 1u;
        ok = wait_inputs(a, (uint64_t)(uintptr_t)x + span, abortp);
        if (ok && mu) ok = wait_inputs(a, (uint64_t)(uintptr_t)xp + span, abortp);
      }
      ok = named_bar_and(5, kStagerThreads, ok);
    }
    if (ok && mu) {
      for (int e = stid; e < (int)ev.segd.mu_entries; e += kStagerThreads) mucb[e] = __ldg(reinterpret_cast<const uint32_t*>(ev.seg.mu_aux) + e);
      named_bar_sync(5, kStagerThreads);
      const int bits = (int)ev.segd.mu_bits;
      const uint32_t mask = (1u << bits) - 1u;
      for (int c8 = stid; c8 < nvr; c8 += kStagerThreads) {
        const int col = col0 + 8 * c8;
        uint4 m = make_uint4(0u, 0u, 0u, 0u);
        if (col < ic) {
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
        const int col = col0 + 8 * c8;
        uint4 r = make_uint4(0u, 0u, 0u, 0u);
        if (col < ic) r = __ldg(reinterpret_cast<const uint4*>(xp + (size_t)b * ic + col));
        *reinterpret_cast<uint4*>(xb + (size_t)b * xstride + (size_t)c8 * 16) = r;
      }
    }
    if (ok && ev.barrier && stid == 0) {
      // grid-wide stage barrier: every CTA has finished (and published) the previous stage.  Each
      // barrier has its own arrival counter, so a CTA without work may run ahead and arrive at
      // later barriers without releasing this one early.
      uint32_t it = 0;
      while ((int)(ld_acquire_gpu(a.counter + (ev.barrier - 1u)) - (a.target + a.wait_skew)) < 0) {
        if (++it >= (a.poll_limit << 2) || *abortp) { *abortp = 1; atomicExch(a.status, (int)RWKVQ_ETIMEOUT); ok = false; break; }
      }
    }
    ok = named_bar_and(6, kStagerThreads, ok);   // uniform verdict; orders the mu row before its readers
    if (ok) {
      float* gs = reinterpret_cast<float*>(xb + (size_t)a.B * xstride);
      for (int v0 = stid; v0 < total; v0 += kStagerThreads * kStageUnroll) {
        uint4 raw[kStageUnroll];
#pragma unroll
        for (int u = 0; u < kStageUnroll; ++u) {
          const int v = v0 + u * kStagerThreads;
          raw[u] = make_uint4(0u, 0u, 0u, 0u);
          if (v < total) {
            const int b = v / nvr, c8 = v - b * nvr;
            const int col = col0 + 8 * c8;
            if (col < ic) raw[u] = __ldcg(reinterpret_cast<const uint4*>(x + (size_t)b * ic + col));
          }
        }
#pragma unroll
        for (int u = 0; u < kStageUnroll; ++u) {
          const int v = v0 + u * kStagerThreads;
          if (v >= total) break;                      // warp-uniform: total is a multiple of 32
          const int b = v / nvr, c8 = v - b * nvr;
          uint4 r = raw[u];
          uint8_t* dst = xb + (size_t)b * xstride + (size_t)c8 * 16;
          if (mu) {
            const uint4 pr = *reinterpret_cast<const uint4*>(dst);          // this thread's own earlier store
            const uint4 mr = *reinterpret_cast<const uint4*>(murow + (size_t)c8 * 16);
            r.x = mix2(r.x, pr.x, mr.x); r.y = mix2(r.y, pr.y, mr.y);
            r.z = mix2(r.z, pr.z, mr.z); r.w = mix2(r.w, pr.w, mr.w);
          }
          *reinterpret_cast<uint4*>(dst) = r;
          if (sums) {
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
    }
    __syncwarp();
    // A stager that gave up still arrives, so that no consumer is left waiting on this barrier;
    // the consumers stop at the abort flag.
    if (lane == 0) mbar_arrive(&ctrl->xfull[buf]);
    ++nseg;
    if (!ok) break;
  }
}

// Six words of one 128-column group of the record of lane `lane` (planes of 512 bytes, 16 bytes
// per lane): group 0 = words 0..5, group 1 = words 6..11.
template <int GRP>
__device__ __forceinline__ void sq_group_words(const uint8_t* rec, int lane, uint32_t (&w)[6]) {
  if constexpr (GRP == 0) {
    const uint4 p0 = *reinterpret_cast<const uint4*>(rec + lane * 16);
    const uint2 p1 = *reinterpret_cast<const uint2*>(rec + 512 + lane * 16);
    w[0] = p0.x; w[1] = p0.y; w[2] = p0.z; w[3] = p0.w; w[4] = p1.x; w[5] = p1.y;
  } else {
    const uint2 p1 = *reinterpret_cast<const uint2*>(rec + 512 + lane * 16 + 8);
    const uint4 p2 = *reinterpret_cast<const uint4*>(rec + 1024 + lane * 16);
    w[0] = p1.x; w[1] = p1.y; w[2] = p2.x; w[3] = p2.y; w[4] = p2.z; w[5] = p2.w;
  }
}

// One 128-column group of the two records of a warp: the input fragments are loaded once and shared
// by both records, whose tensor-core chains run interleaved.
template <int NB, int GRP>
__device__ __forceinline__ void sq_pair(const uint32_t (&wa)[6], const uint32_t (&wb)[6], const uint4 sza, const uint4 szb,
                                        bool has_b, const XLane& xl, float (&acca)[NB][4], float (&accb)[NB][4]) {
  sq_group_mma2<NB, GRP>(wa, wb, sza, szb, has_b, xl, acca, accb);
}

template <int BITS, int NB, int HALF>
__device__ __forceinline__ void vq_pair(const uint32_t (&wa)[2 * BITS], const uint32_t (&wb)[2 * BITS], const uint32_t* cb_lane,
                                        const XLane& xl, float (&acca)[NB][4], float (&accb)[NB][4]) {
  vq_half_mma2<BITS, NB, HALF>(wa, wb, cb_lane, xl, acca, accb);
}

// c[k] of the four lanes whose row index g differs in its two low bits (lanes 4 apart) -> lane i (= g & 3)
// ends with element i of lanes g & ~3 ... (g & ~3) + 3, in that order.  All lanes of the warp call it.
__device__ __forceinline__ void transpose4_lanes(float (&c)[4], int i) {
  const bool hi = (i & 2) != 0, lo = (i & 1) != 0;
  const float s0 = hi ? c[0] : c[2], s1 = hi ? c[1] : c[3];
  const float r0 = __shfl_xor_sync(0xFFFFFFFFu, s0, 8), r1 = __shfl_xor_sync(0xFFFFFFFFu, s1, 8);
  // element 2*hi + {0, 1} of source lanes j1 = 0, 1
  const float a00 = hi ? r0 : c[0], a01 = hi ? r1 : c[1];
  const float a10 = hi ? c[2] : r0, a11 = hi ? c[3] : r1;
  const float q0 = lo ? a00 : a01, q1 = lo ? a10 : a11;
  const float p0 = __shfl_xor_sync(0xFFFFFFFFu, q0, 4), p1 = __shfl_xor_sync(0xFFFFFFFFu, q1, 4);
  c[0] = lo ? p0 : a00;  c[1] = lo ? a01 : p0;
  c[2] = lo ? p1 : a10;  c[3] = lo ? a11 : p1;
}
__device__ __forceinline__ void red_add_v4(float* p, const float (&v)[4]) {
  asm volatile("red.global.v4.f32.add [%0], {%1, %2, %3, %4};" :: "l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
}

// Consumer warp `w` of group `grp`: units grp, grp + 2, ... of the CTA's list.
template <int NB, bool MIX>
__device__ void consumer_role(const StepArgs& a, uint8_t* smem, Ctrl* ctrl, const uint8_t* xbufs, uint8_t* replicas,
                              uint32_t unit_base, uint32_t n_units, uint32_t ev_base, uint32_t n_events) {
  bool dead = false;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kGroups = Shape<NB>::kGroups;
  const int grp = warp >> 3, w = warp & 7;
  const int g = lane >> 2, t = lane & 3;
  volatile int* abortp = &ctrl->abort_flag;
  float acca[NB][4], accb[NB][4];
#pragma unroll
  for (int n = 0; n < NB; ++n)
#pragma unroll
    for (int k = 0; k < 4; ++k) acca[n][k] = accb[n][k] = 0.f;
  // Every consumer warp walks the CTA's event list in order -- it reports each stage it leaves and
  // passes through each input segment, used or not -- so that the phases of the shared barriers
  // advance in step for all consumer warps.
  int held = -1;              // input segment this warp currently holds
  uint32_t seg_next = 0;      // number of segment events passed so far
  uint32_t cur_ev = 0;        // last event processed (event 0 is the clearing arrival: nothing to do)
  // Report the current stage as finished (stage_report).  The lanes' reductions into y are ordered
  // before lane 0's report by the warp barrier; no lane fences at GPU scope itself: that would only
  // add its latency to the end of every stage.
  uint32_t next_bar = 1u;     // every CTA arrives at barriers 1, 2, ... in this order, once per stage
  auto arrive_stage = [&]() {
    __syncwarp();
    if constexpr (NB == 2) {
      if (lane == 0 && !dead) stage_report_total(ctrl, next_bar);
      ++next_bar;
    } else {
      if (lane == 0 && !dead) stage_report<NB>(ctrl, a, next_bar);
      ++next_bar;
    }
  };
  auto release_held = [&]() {
    __syncwarp();
    if (held >= 0 && lane == 0 && !dead) mbar_arrive(&ctrl->xempty[(uint32_t)held % XBufs<MIX, NB>::kCount]);
    held = -1;
  };
  auto pass_segment = [&]() {   // a segment this warp does not use: observe it, hand it back
    const uint32_t q = seg_next++;
    if (!dead && !mbar_wait_warp(&ctrl->xfull[q % XBufs<MIX, NB>::kCount], (q / XBufs<MIX, NB>::kCount) & 1u, abortp, a.status)) dead = true;
    __syncwarp();
    if (lane == 0 && !dead) mbar_arrive(&ctrl->xempty[q % XBufs<MIX, NB>::kCount]);
  };
  // Events (cur_ev, upto) in order; `mask` describes them when there are at most 32 and the planner
  // could say so, otherwise (and for the tail of the list) the kinds are read from the plan, 32 at
  // a time.
  auto pass_events = [&](uint32_t upto, uint32_t mask, bool mask_valid) {
    if (cur_ev + 1u >= upto) return;
    release_held();
    while (cur_ev + 1u < upto && !dead) {
      const uint32_t first = cur_ev + 1u;
      const uint32_t cnt = min(32u, upto - first);
      uint32_t m = mask;
      if (!mask_valid) {
        bool arr = false;
        if ((uint32_t)lane < cnt) {
          const uint2 kb = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint8_t*>(a.events) + (size_t)(ev_base + first + lane) * 64 + 48));
          arr = kb.x == EV_ARRIVE && kb.y > 0u;
        }
        m = __ballot_sync(0xFFFFFFFFu, arr);
      }
      for (uint32_t j = 0; j < cnt && !dead; ++j) {
        if ((m >> j) & 1u) arrive_stage(); else pass_segment();
      }
      cur_ev += cnt;
      mask_valid = false;
    }
  };
  uint8_t* rep = replicas + (size_t)grp * a.replica_bytes;
  // slot and round of unit i (i % n_slots, i / n_slots), advanced without dividing
  const uint32_t n_slots_u = (uint32_t)a.n_slots;
  uint32_t slot_u = (uint32_t)grp % n_slots_u, round = (uint32_t)grp / n_slots_u;
  for (uint32_t i = (uint32_t)grp; i < n_units; i += kGroups, slot_u += kGroups) {
    while (slot_u >= n_slots_u) { slot_u -= n_slots_u; ++round; }
    const int slot = (int)slot_u;
    const uint8_t* sl = smem + kCtrlBytes + (size_t)slot * a.slot_bytes;
    const StepUnit* u = reinterpret_cast<const StepUnit*>(sl);
    if (!dead && !mbar_wait_warp(&ctrl->full[slot], round & 1u, abortp, a.status)) dead = true;
    if (!dead && u->ev_index != cur_ev) {
      const uint32_t target = u->ev_index;
      pass_events(target, u->between_mask, target - cur_ev - 1u <= 32u);
      if (!dead) {
        release_held();
        const uint32_t q = seg_next++;
        held = (int)q;
        cur_ev = target;
        if (!mbar_wait_warp(&ctrl->xfull[q % XBufs<MIX, NB>::kCount], (q / XBufs<MIX, NB>::kCount) & 1u, abortp, a.status)) dead = true;
      }
    }
    if (dead) {
      // A warp that gave up keeps walking the list only to keep the group's named barriers whole
      // (the other warps stop at their next bounded wait); it touches neither slots nor outputs.
      if (a.units[unit_base + i].flags & UF_VQ) { named_bar_sync(1 + grp, kGroupThreads); named_bar_sync(1 + grp, kGroupThreads); }
      continue;
    }
    const uint32_t flags = u->flags;
    const uint32_t by1 = u->bytes1;
    const uint32_t after_count = u->after_count, after_mask = u->after_mask;
    const uint8_t* data = sl + 128;
    const uint8_t* xb = xbufs + (size_t)((uint32_t)held % XBufs<MIX, NB>::kCount) * XBufs<MIX, NB>::kBytes;
    const uint32_t xstride = u->xstride, nbp = u->nbp, chb = u->chunk_bytes, rb = u->rec_bytes;
    const uint32_t w0 = (flags >> 8) & 15u, w1 = (flags >> 12) & 15u;
    const bool active = (uint32_t)w >= w0 && (uint32_t)w < w1;
    const bool has_b = by1 != 0u;
    const uint32_t oc = u->oc, row0 = u->row0;
    float* y = reinterpret_cast<float*>(u->y);
    const uint8_t* ra = data + (size_t)w * rb;
    const uint8_t* rbp = data + chb + (size_t)w * rb;
    if (!(flags & UF_VQ)) {
      const uint32_t col = u->xcol0;
      const XLane xl = make_xlane(xb + (size_t)col * 2, xstride,
                                  reinterpret_cast<const float*>(xb + u->gs_off) + (size_t)(col >> 7) * 3 * nbp, nbp, a.B, lane);
      if constexpr (NB == 2) {
        // Registers suffice for the whole record pair: take all of it, free the slot, then run both
        // 128-column groups as one stretch of code (eight tensor-core chains for the scheduler to interleave).
        uint32_t wa0[6], wb0[6], wa1[6], wb1[6];
        uint4 sza = make_uint4(0, 0, 0, 0), szb = sza;
        if (active) {
          sq_group_words<0>(ra, lane, wa0);
          sq_group_words<1>(ra, lane, wa1);
          sza = *reinterpret_cast<const uint4*>(ra + RWKVQ_SQ_CODE_BYTES + g * 16);
          if (has_b) {
            sq_group_words<0>(rbp, lane, wb0);
            sq_group_words<1>(rbp, lane, wb1);
            szb = *reinterpret_cast<const uint4*>(rbp + RWKVQ_SQ_CODE_BYTES + g * 16);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctrl->empty[slot]);
        if (active) {
          sq_pair<NB, 0>(wa0, wb0, sza, szb, has_b, xl, acca, accb);
          sq_pair<NB, 1>(wa1, wb1, sza, szb, has_b, xl, acca, accb);
        }
      } else {
      uint32_t wa[6], wb[6];
      uint4 sza = make_uint4(0, 0, 0, 0), szb = sza;
      if (active) {
        sq_group_words<0>(ra, lane, wa);
        sza = *reinterpret_cast<const uint4*>(ra + RWKVQ_SQ_CODE_BYTES + g * 16);
        if (has_b) {
          sq_group_words<0>(rbp, lane, wb);
          szb = *reinterpret_cast<const uint4*>(rbp + RWKVQ_SQ_CODE_BYTES + g * 16);
        }
        sq_pair<NB, 0>(wa, wb, sza, szb, has_b, xl, acca, accb);
        sq_group_words<1>(ra, lane, wa);
        if (has_b) sq_group_words<1>(rbp, lane, wb);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl->empty[slot]);     // the rest of the records is in registers: free the slot
      if (active) sq_pair<NB, 1>(wa, wb, sza, szb, has_b, xl, acca, accb);
      }
    } else {
      // replicate the tile's codebook for conflict-free lookups (the eight warps of the group)
      const uint32_t E = u->entries;
      named_bar_sync(1 + grp, kGroupThreads);          // the group's previous lookups are done
      {
        const uint32_t* cbraw = reinterpret_cast<const uint32_t*>(data + 2 * chb);
        uint32_t* rp = reinterpret_cast<uint32_t*>(rep);
        for (uint32_t idx = (uint32_t)(w * 32 + lane); idx < E * 32u; idx += kGroupThreads) rp[idx] = cbraw[idx >> 5];
      }
      named_bar_sync(1 + grp, kGroupThreads);
      const uint32_t* cb_lane = reinterpret_cast<const uint32_t*>(rep) + lane;
      const XLane xl = make_xlane(xb + (size_t)u->xcol0 * 2, xstride, nullptr, nbp, a.B, lane);
      if (flags & UF_BITS8) {
        uint32_t va[16], vb[16];
        if (active) {
          vq_half_words<8, 0>(ra, lane, va); vq_half_words<8, 0>(rbp, lane, vb);
          vq_pair<8, NB, 0>(va, vb, cb_lane, xl, acca, accb);
          vq_half_words<8, 1>(ra, lane, va); vq_half_words<8, 1>(rbp, lane, vb);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctrl->empty[slot]);
        if (active) vq_pair<8, NB, 1>(va, vb, cb_lane, xl, acca, accb);
      } else {
        uint32_t va[12], vb[12];
        if (active) {
          vq_half_words<6, 0>(ra, lane, va); vq_half_words<6, 0>(rbp, lane, vb);
          vq_pair<6, NB, 0>(va, vb, cb_lane, xl, acca, accb);
          vq_half_words<6, 1>(ra, lane, va); vq_half_words<6, 1>(rbp, lane, vb);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctrl->empty[slot]);
        if (active) vq_pair<6, NB, 1>(va, vb, cb_lane, xl, acca, accb);
      }
    }
    if (flags & UF_FLUSH) {
      if (active) {
        {
          // Four lanes that share t hold a 4 x 4 block (rows 4J .. 4J+3 of one row half x the accumulator's four
          // elements): transposed, every lane owns four consecutive rows of ONE batch column and adds them
          // with a single 16-byte reduction instead of four scattered ones.  The plan accepts only outputs
          // that start on a 16-byte boundary, and the format only row counts that are multiples of 16.
          const int i = g & 3;
          const uint32_t rbase = row0 + (uint32_t)w * 16u + 8u * (uint32_t)(i >> 1) + (uint32_t)(g & ~3);
#pragma unroll
          for (int n = 0; n < NB; ++n) {
            const int b = n * 8 + 2 * t + (i & 1);
            float va[4] = {acca[n][0], acca[n][1], acca[n][2], acca[n][3]};
            transpose4_lanes(va, i);
            if (b < a.B && rbase < oc) red_add_v4(y + (size_t)b * oc + rbase, va);
            if (has_b) {                      // warp-uniform
              float vb[4] = {accb[n][0], accb[n][1], accb[n][2], accb[n][3]};
              transpose4_lanes(vb, i);
              if (b < a.B && rbase + 128u < oc) red_add_v4(y + (size_t)b * oc + rbase + 128u, vb);
            }
          }
        }
      }
#pragma unroll
      for (int n = 0; n < NB; ++n)
#pragma unroll
        for (int k = 0; k < 4; ++k) acca[n][k] = accb[n][k] = 0.f;
    }
    // the group's last unit of the stage: report the stage as finished without waiting for the next unit
    if (after_count) pass_events(cur_ev + after_count + 1u, after_mask, true);
  }
  if (!dead) {
    release_held();
    pass_events(n_events, 0u, false);     // the rest of the list: later stages this warp has no unit in
  }
}

template <int NB, bool MIX>
__global__ void __launch_bounds__(Shape<NB>::kThreads, 1) step_kernel(const StepArgs a) {
  constexpr int kConsumerWarps = Shape<NB>::kConsumerWarps, kStagerWarps = Shape<NB>::kStagerWarps;
  extern __shared__ __align__(128) uint8_t smem[];
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem);
  uint8_t* xbufs = smem + kCtrlBytes + (size_t)a.n_slots * a.slot_bytes;
  uint32_t* mucb = reinterpret_cast<uint32_t*>(xbufs + kXBufTotal);
  uint8_t* replicas = reinterpret_cast<uint8_t*>(mucb) + kMuScratch;
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.n_slots; ++s) { mbar_init(&ctrl->full[s], 1); mbar_init(&ctrl->empty[s], kGroupWarps); }
    for (int b = 0; b < 4; ++b) { mbar_init(&ctrl->xfull[b], kStagerWarps); mbar_init(&ctrl->xempty[b], kConsumerWarps); }
    for (int k = 0; k < 64; ++k) ctrl->stage_cnt[k] = 0u;
    ctrl->abort_flag = 0;
    ctrl->poll_limit = (int)a.poll_limit;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const uint32_t u0 = a.unit_off[blockIdx.x], u1 = a.unit_off[blockIdx.x + 1];
  const uint32_t e0 = a.event_off[blockIdx.x], e1 = a.event_off[blockIdx.x + 1];
  const int warp = threadIdx.x >> 5;
  // Registers are re-divided at entry (see Shape): the warpgroups of stagers and producer hand part of
  // their share back and the consumer warpgroups take it, so that the record routine keeps everything
  // in registers.
  if (warp < kConsumerWarps) {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" :: "n"(Shape<NB>::kConsumerRegs));
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" :: "n"(Shape<NB>::kStagerRegs));
  }
  if (warp < kConsumerWarps) {
    consumer_role<NB, MIX>(a, smem, ctrl, xbufs, replicas, u0, u1 - u0, e0, e1 - e0);
  } else if (warp < kConsumerWarps + kStagerWarps) {
    stager_role<MIX, NB>(a, smem, ctrl, xbufs, mucb, e0, e1);
  } else {
    producer_role(a, smem, ctrl, u0, u1);
  }
}

// ---- host planner --------------------------------------------------------------------------------

struct PlanInfo {
  int P, B, NB, n_slots, n_stages, mix;
  unsigned runs;        // launches since the counters were last zero
  unsigned abort_epoch; // value of the abort epoch when the counters were last known good
  uint32_t poll_limit, wait_skew;
  uint32_t slot_bytes, replica_bytes, smem_bytes;
  size_t off_unit_off, off_event_off, off_units, off_events, off_counter, off_mixops, off_mixx, off_scratch, total_bytes;
  uint32_t n_units, n_events, n_barriers;
  std::vector<uint64_t> y_lo, y_hi;   // per stage: device address range its products write (host-buffer runs)
};

static std::mutex g_plan_mutex;
static std::unordered_map<const void*, PlanInfo> g_plans;

struct HostUnit {
  StepUnit u;
  int op, tr, kt, stage, w0, w1;
};

// Shared-memory footprint of an input segment: B rows of x_mix, the per-group sums (SQ) and one
// row of decoded mu_hat (products with a token shift).
static uint32_t xseg_mu_off(int B, int ncols, bool sums) {
  uint32_t xstride = (uint32_t)ncols * 2u + 32u;
  uint32_t nbp = (uint32_t)((B + 1) & ~1);
  // 64 bytes of slack: lanes of batch columns that do not exist read (and discard) sums past the table
  uint32_t off = (uint32_t)B * xstride + (sums ? (uint32_t)(ncols / 128) * 3u * nbp * 4u + 64u : 0u);
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
    if (!o.W_image_dev || !o.y_dev) return RWKVQ_EINVAL;
    const rwkvq_input_xform& in = o.in;
    if (in.kind == RWKVQ_IN_BUFFER) {
      if (!o.x_fp16_dev) return RWKVQ_EINVAL;
    } else {
      if (in.kind != RWKVQ_IN_WKV && in.kind != RWKVQ_IN_RELU2 && in.kind != RWKVQ_IN_F32) return RWKVQ_EINVAL;
      if (!in.src_f32 || !aligned16(in.src_f32)) return in.src_f32 ? RWKVQ_EALIGN : RWKVQ_EINVAL;
      if (in.kind == RWKVQ_IN_WKV) {
        const void* need[] = {in.k_f32, in.v_f32, in.state_a, in.state_b, in.state_p, in.u_f32, in.w_f32};
        for (const void* q : need) {
          if (!q) return RWKVQ_EINVAL;
          if (!aligned16(q)) return RWKVQ_EALIGN;
        }
      }
      if (in.kind == RWKVQ_IN_F32 && in.gate_f32 && !aligned16(in.gate_f32)) return RWKVQ_EALIGN;
      if (in.flags & ~RWKVQ_INF_RMSNORM) return RWKVQ_EINVAL;
      if ((in.flags & RWKVQ_INF_RMSNORM) && (in.kind != RWKVQ_IN_F32 || o.W_desc.ic % 64)) return RWKVQ_EUNSUPPORTED;
      if (o.W_desc.ic % 8) return RWKVQ_ESHAPE;
    }
    if (in.xprev_out_fp16 && !aligned16(in.xprev_out_fp16)) return RWKVQ_EALIGN;
    if ((o.mu_image_dev == nullptr) != (o.xprev_fp16_dev == nullptr)) return RWKVQ_EINVAL;
    if (o.mu_image_dev) {
      st = check_vector_desc(&o.mu_desc, o.W_desc.ic);
      if (st != RWKVQ_OK) return st;
      if (!aligned16(o.mu_image_dev) || !aligned16(o.xprev_fp16_dev)) return RWKVQ_EALIGN;
    }
    if (!aligned16(o.W_image_dev) || (o.x_fp16_dev && !aligned16(o.x_fp16_dev)) || !aligned16(o.y_dev)) return RWKVQ_EALIGN;
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
  const int kGroups = groups_of(B <= 8 ? 1 : 2);   // consumer groups per CTA: they take a CTA's units in turn
  uint32_t data_max = 0;
  if (has_sq) data_max = std::max(data_max, 2u * 8u * RWKVQ_SQ_RECORD_BYTES);
  if (has_vq6) data_max = std::max(data_max, 2u * 8u * 1536u + 256u);
  if (has_vq8) data_max = std::max(data_max, 2u * 8u * 2048u + 1024u);
  info->slot_bytes = (128u + data_max + 127u) & ~127u;
  info->replica_bytes = has_vq8 ? 256u * 128u : has_vq6 ? 64u * 128u : 0u;   // per consumer group
  const uint32_t fixed = kCtrlBytes + kXBufTotal + kMuScratch + (uint32_t)kGroups * info->replica_bytes;
  int ns = (int)((kSmemLimit - fixed) / info->slot_bytes);
  if (ns > kMaxSlots) ns = kMaxSlots;
  if (ns < 2) return RWKVQ_EUNSUPPORTED;
  info->n_slots = ns;
  info->smem_bytes = fixed + (uint32_t)ns * info->slot_bytes;
  info->P = P; info->B = B; info->NB = B <= 8 ? 1 : 2;
  info->poll_limit = kDefaultPollLimit; info->wait_skew = 0;
  bool any_xform = false;
  for (int i = 0; i < n_ops; ++i) any_xform = any_xform || ops[i].in.kind != RWKVQ_IN_BUFFER || ops[i].in.xprev_out_fp16 != nullptr;
  // see StepArgs::mix; the element-wise operators in front of a product exist in the stage pre-pass only
  const bool mix = B >= 4 || any_xform;
  const uint32_t xbuf_bytes = XBufs<false, 1>::kBytes;
  info->mix = mix ? 1 : 0;
  const uint32_t nbp = (uint32_t)((B + 1) & ~1);

  std::vector<std::pair<int, int>> stage_ranges;  // [first op, last op) per distinct stage value
  for (int i = 0; i < n_ops;) {
    int j = i;
    while (j < n_ops && ops[j].stage == ops[i].stage) ++j;
    stage_ranges.push_back({i, j});
    i = j;
  }
  const int n_stages = (int)stage_ranges.size();
  if ((uint32_t)n_stages + 1u > kMaxBarriers) return RWKVQ_EUNSUPPORTED;   // per-barrier counts in the control block
  info->n_stages = n_stages;
  info->n_barriers = ((uint32_t)n_stages + 1) * (mix ? 2u : 1u);   // the pre-pass has a barrier of its own per stage

  std::vector<std::vector<HostUnit>> cta_units(P);
  std::vector<std::vector<StepEvent>> cta_arrivals(P);      // arrival events, one per barrier
  bool too_many_ranges = false;
  auto make_arrival = [&](int c, int stage_idx_to_clear, int barrier) {
    StepEvent ev;
    std::memset(&ev, 0, sizeof(ev));
    ev.kind = EV_ARRIVE; ev.barrier = (uint32_t)barrier;
    if (stage_idx_to_clear < n_stages) {
      uint64_t total = 0;
      for (int o = stage_ranges[stage_idx_to_clear].first; o < stage_ranges[stage_idx_to_clear].second; ++o)
        total += (uint64_t)B * ops[o].W_desc.oc;
      const uint64_t lo = total * (uint64_t)c / P, hi = total * (uint64_t)(c + 1) / P;
      uint64_t base = 0;
      int k = 0;
      for (int o = stage_ranges[stage_idx_to_clear].first; o < stage_ranges[stage_idx_to_clear].second; ++o) {
        const uint64_t n = (uint64_t)B * ops[o].W_desc.oc;
        const uint64_t a0 = std::max(lo, base), a1 = std::min(hi, base + n);
        if (a1 > a0) {
          if (k >= 3) { too_many_ranges = true; break; }
          ev.arr.zptr[k] = (uint64_t)(uintptr_t)ops[o].y_dev + (a0 - base) * 4;
          ev.arrd.zcount[k] = (uint32_t)(a1 - a0);
          ++k;
        }
        base += n;
      }
    }
    if (mix && barrier < n_stages) {
      // this CTA's share of the pre-pass of stage `barrier`
      uint64_t G = 0;
      for (int o = stage_ranges[barrier].first; o < stage_ranges[barrier].second; ++o) G += (uint64_t)B * (ops[o].W_desc.ic_pad / 128);
      ev.arr.grp_lo = (uint32_t)(G * (uint64_t)c / P); ev.arr.grp_hi = (uint32_t)(G * (uint64_t)(c + 1) / P);
      ev.arrd.op_first = (uint16_t)stage_ranges[barrier].first;
      ev.arrd.op_count = (uint16_t)(stage_ranges[barrier].second - stage_ranges[barrier].first);
    }
    cta_arrivals[c].push_back(ev);
  };
  for (int c = 0; c < P; ++c) make_arrival(c, 0, 0);   // barrier 0: the first stage's outputs are clear

  for (int s = 0; s < n_stages; ++s) {
    std::vector<HostUnit> units;
    for (int o = stage_ranges[s].first; o < stage_ranges[s].second; ++o) {
      const rwkvq_desc& d = ops[o].W_desc;
      const uint8_t* img = static_cast<const uint8_t*>(ops[o].W_image_dev);
      const uint8_t* payload = img + RWKVQ_HEADER_BYTES;
      const int KT = d.ic_pad / 256, MB = d.oc_pad / 128;
      const bool vq = d.method != RWKVQ_SQ;
      const uint32_t rb = vq ? rwkvq_vq_record_bytes(d.bits) : (uint32_t)RWKVQ_SQ_RECORD_BYTES;
      const uint32_t cb = 8u * rb;
      const uint8_t* aux = vq ? img + matrix_aux_offset(&d) : nullptr;
      for (int tr = 0; tr < (MB + 1) / 2; ++tr)
        for (int kt = 0; kt < KT; ++kt) {
          HostUnit h;
          std::memset(&h, 0, sizeof(h));
          h.u.flags = vq ? (UF_VQ | (d.bits == 8 ? UF_BITS8 : 0)) : 0;
          h.u.src0 = (uint64_t)(uintptr_t)(payload + (size_t)((2 * tr) * KT + kt) * cb);
          h.u.bytes0 = cb;
          if (2 * tr + 1 < MB) { h.u.src1 = (uint64_t)(uintptr_t)(payload + (size_t)((2 * tr + 1) * KT + kt) * cb); h.u.bytes1 = cb; }
          if (vq) {
            h.u.cb_src = (uint64_t)(uintptr_t)(aux + (size_t)(tr * KT + kt) * d.entries * 4);
            h.u.cb_bytes = (uint32_t)d.entries * 4u; h.u.entries = (uint32_t)d.entries;
          }
          h.u.chunk_bytes = cb; h.u.rec_bytes = rb;
          h.u.row0 = (uint32_t)tr * 256u; h.u.oc = (uint32_t)d.oc; h.u.y = (uint64_t)(uintptr_t)ops[o].y_dev;
          h.u.stage = (uint32_t)s;
          h.op = o; h.tr = tr; h.kt = kt; h.stage = s;
          units.push_back(h);
        }
    }
    // contiguous, cost-balanced ranges cut at one eighth of a unit (the records of one warp).  The
    // cost of a unit is its record count weighted by what a record of its format costs the consumer
    // warps (measured with every product in one stage: a VQ record with 64 entries takes about 1.45
    // times, one with 256 entries about 1.25 times as long as an SQ record), so that the CTAs that
    // get a stage's VQ matrix do not finish last.
    auto cost_of = [&](const HostUnit& h) -> uint64_t {
      const uint64_t recs = (h.u.bytes0 + h.u.bytes1) / h.u.rec_bytes;
      // in twentieths of an SQ record; the table lookups weigh more the more batch columns a record meets
      // (whole-step times of all-SQ against all-VQ-64 stacks less the per-stage chain: 1.4 at B = 1,
      // 1.6 at B = 8, 2.0 at B = 16)
      const uint64_t vq6 = B > 8 ? 40u : B >= 4 ? 32u : 29u, vq8 = B > 8 ? 34u : B >= 4 ? 28u : 25u;
      const uint64_t wgt = !(h.u.flags & UF_VQ) ? 20u : (h.u.flags & UF_BITS8) ? vq8 : vq6;
      return recs * wgt * 64u;
    };
    // A consumer group spends about the same time on a piece of a unit as on a whole unit (the
    // warps without a record idle), and every further input segment of a CTA costs about 1.7 us of
    // serial staging; traces of all CTAs' barrier arrivals showed the stages waiting for the CTAs
    // with the most pieces and segments, not for the most bytes.  So units are dealt WHOLE, and
    // where it balances, row by row: each row of tiles (one product, one 256-row block: one input
    // segment) gets a number of CTAs, greedily the row with the largest cost per CTA first, and
    // its units are split into that many runs of neighbouring column tiles.  This is taken when no
    // CTA ends up more than one unit above the even share; small stages leave some CTAs idle.
    bool dealt = false;
    auto push_whole = [&](int c, const HostUnit& h) {
      HostUnit part = h;
      part.w0 = 0; part.w1 = 8;
      part.u.off0 = 0;
      part.u.flags |= (0u << 8) | (8u << 12);
      cta_units[c].push_back(part);
    };
    {
      struct Row { size_t first, count; uint64_t cost; int k; };
      std::vector<Row> rows;
      for (size_t i = 0; i < units.size();) {
        size_t j = i;
        uint64_t cst = 0;
        while (j < units.size() && units[j].op == units[i].op && units[j].tr == units[i].tr) { cst += cost_of(units[j]); ++j; }
        rows.push_back(Row{i, j - i, cst, 1});
        i = j;
      }
      if (!rows.empty() && rows.size() <= (size_t)P) {
        int spare = P - (int)rows.size();
        while (spare > 0) {
          size_t best = rows.size();
          uint64_t best_cost = 0;
          for (size_t r = 0; r < rows.size(); ++r) {
            if ((size_t)rows[r].k >= rows[r].count) continue;          // one unit per CTA at most
            const uint64_t per = rows[r].cost / (uint64_t)rows[r].k;
            if (per > best_cost) { best_cost = per; best = r; }
          }
          if (best == rows.size()) break;
          ++rows[best].k; --spare;
        }
        size_t max_units = 0;
        for (const Row& r : rows) max_units = std::max(max_units, (r.count + (size_t)r.k - 1) / (size_t)r.k);
        const size_t even = (units.size() + (size_t)P - 1) / (size_t)P;
        if (max_units <= even + 1) {
          // start at a CTA that moves with the stage, so that idle CTAs are not always the same SMs
          size_t c = ((size_t)s * 37u) % (size_t)P;
          for (const Row& r : rows)
            for (int q = 0; q < r.k; ++q) {
              const size_t lo = r.count * (size_t)q / (size_t)r.k, hi = r.count * (size_t)(q + 1) / (size_t)r.k;
              for (size_t i = lo; i < hi; ++i) push_whole((int)c, units[r.first + i]);
              c = (c + 1) % (size_t)P;
            }
          dealt = true;
        }
      }
    }
    uint64_t total = 0;
    for (const HostUnit& h : units) total += cost_of(h);
    uint64_t run = 0;
    auto cta_of = [&](uint64_t mid) {
      int c = (int)((mid * (uint64_t)P) / (total ? total : 1));
      return c >= P ? P - 1 : c;
    };
    const bool whole_units = units.size() >= (size_t)4 * (size_t)P;   // many units per CTA: a whole unit at its cost midpoint
    for (const HostUnit& h : units) {
      if (dealt) break;
      if (whole_units) {
        push_whole(cta_of(run + cost_of(h) / 2), h);
        run += cost_of(h);
        continue;
      }
      const uint64_t e8 = cost_of(h) / 8;
      int w = 0;
      while (w < 8) {
        const int c = cta_of(run + (uint64_t)w * e8 + e8 / 2);
        int w1 = w + 1;
        while (w1 < 8 && cta_of(run + (uint64_t)w1 * e8 + e8 / 2) == c) ++w1;
        HostUnit part = h;
        part.w0 = w; part.w1 = w1;
        const uint32_t rb = h.u.rec_bytes;
        part.u.off0 = (uint32_t)w * rb;
        part.u.src0 = h.u.src0 + (uint64_t)w * rb;
        part.u.bytes0 = (uint32_t)(w1 - w) * rb;
        if (h.u.bytes1) { part.u.src1 = h.u.src1 + (uint64_t)w * rb; part.u.bytes1 = (uint32_t)(w1 - w) * rb; }
        part.u.flags |= ((uint32_t)w << 8) | ((uint32_t)w1 << 12);
        cta_units[c].push_back(part);
        w = w1;
      }
      run += cost_of(h);
    }
    for (int c = 0; c < P; ++c) make_arrival(c, s + 1, s + 1);
  }
  if (too_many_ranges) return RWKVQ_EUNSUPPORTED;   // a CTA's slice of a stage's outputs may touch at most three products

  // pre-pass outputs: one region, reused by every stage (a stage's pre-pass starts only after the
  // previous stage, and with it every copy out of the region, has finished everywhere)
  std::vector<uint64_t> mix_x_off(n_ops, 0), mix_sums_off(n_ops, 0);
  std::vector<StepMixOp> mixops(mix ? n_ops : 0);
  std::vector<StepMixX> mixx(mix ? n_ops : 0);
  uint64_t scratch_bytes = 0;
  if (mix) {
    for (int st_i = 0; st_i < n_stages; ++st_i) {
      uint64_t off = 0;
      for (int o = stage_ranges[st_i].first; o < stage_ranges[st_i].second; ++o) {
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
        m.kind = (uint16_t)(op.in.kind | ((op.in.kind == RWKVQ_IN_F32 && (op.in.flags & RWKVQ_INF_RMSNORM)) ? 0x100 : 0) |
                            (op.in.xprev_out_fp16 ? 0x200 : 0));
        StepMixX& mx = mixx[o];
        std::memset(&mx, 0, sizeof(mx));
        mx.src = (uint64_t)(uintptr_t)op.in.src_f32;
        mx.k = (uint64_t)(uintptr_t)(op.in.kind == RWKVQ_IN_F32 ? op.in.gate_f32 : op.in.k_f32);
        mx.v = (uint64_t)(uintptr_t)op.in.v_f32;
        mx.state_a = (uint64_t)(uintptr_t)op.in.state_a; mx.state_b = (uint64_t)(uintptr_t)op.in.state_b;
        mx.state_p = (uint64_t)(uintptr_t)op.in.state_p;
        mx.u = (uint64_t)(uintptr_t)op.in.u_f32; mx.w = (uint64_t)(uintptr_t)op.in.w_f32;
        mx.xprev_out = (uint64_t)(uintptr_t)op.in.xprev_out_fp16;
        mx.scale = (uint64_t)(uintptr_t)op.in.scale_f32;
        m.dst_x = mix_x_off[o]; m.dst_sums = mix_sums_off[o];
        m.ic = (uint32_t)op.W_desc.ic; m.ic_pad = (uint32_t)op.W_desc.ic_pad;
        m.sums = op.W_desc.method == RWKVQ_SQ ? 1 : 0;
      }
      bool stage_norm = false;
      for (int o = stage_ranges[st_i].first; o < stage_ranges[st_i].second; ++o) stage_norm = stage_norm || (mixops[o].kind & 0x100);
      if (stage_norm) mixops[stage_ranges[st_i].first].kind |= 0x400;
      bool stage_plain = true;
      for (int o = stage_ranges[st_i].first; o < stage_ranges[st_i].second; ++o) stage_plain = stage_plain && mixops[o].kind == 0;
      if (stage_plain) mixops[stage_ranges[st_i].first].kind |= 0x800;
      scratch_bytes = std::max(scratch_bytes, off);
    }
  }
  std::vector<uint32_t> unit_off(P + 1, 0), event_off(P + 1, 0);
  std::vector<StepUnit> all_units;
  std::vector<StepEvent> all_events;
  for (int c = 0; c < P; ++c) {
    std::vector<HostUnit>& L = cta_units[c];
    unit_off[c] = (uint32_t)all_units.size();
    event_off[c] = (uint32_t)all_events.size();
    const size_t n = L.size();
    // a group accumulates along K in registers while its consecutive units stay on the same rows
    for (size_t i = 0; i < n; ++i) {
      const size_t j = i + (size_t)kGroups;
      const bool same_run = j < n && L[j].stage == L[i].stage && L[j].op == L[i].op && L[j].tr == L[i].tr &&
                            L[j].w0 == L[i].w0 && L[j].w1 == L[i].w1;
      if (!same_run) L[i].u.flags |= UF_FLUSH;
    }
    all_events.push_back(cta_arrivals[c][0]);
    uint32_t seg_no = 0;
    size_t i = 0;
    for (int s = 0; s < n_stages; ++s) {
      // segments: maximal runs of units of one product whose column span fits the buffer
      while (i < n && L[i].stage == s) {
        const int op = L[i].op;
        const bool sums = ops[op].W_desc.method == RWKVQ_SQ;
        const bool has_mu = !mix && ops[op].mu_image_dev != nullptr;   // copied segments carry no mu row
        int kmin = L[i].kt, kmax = L[i].kt + 1;
        size_t j = i + 1, last = i;
        // A segment is a contiguous run of column tiles (a range that wraps from the end of one row
        // pair to the start of the next starts a new segment) that fits the buffer.
        while (j < n && L[j].op == op && L[j].stage == s) {
          if (L[j].kt < kmin || L[j].kt > kmax) break;
          const int nmax = std::max(kmax, L[j].kt + 1);
          if (xseg_bytes(B, (nmax - kmin) * 256, sums, has_mu) > xbuf_bytes) break;
          kmax = nmax; last = j; ++j;
        }
        const int ncols = (kmax - kmin) * 256;
        if (xseg_bytes(B, ncols, sums, has_mu) > xbuf_bytes) return RWKVQ_EUNSUPPORTED;
        StepEvent ev;
        std::memset(&ev, 0, sizeof(ev));
        const rwkvq_gemv_op& o = ops[op];
        ev.kind = EV_SEGMENT;
        ev.seg.x = (uint64_t)(uintptr_t)o.x_fp16_dev;
        ev.segd.ic = (uint32_t)o.W_desc.ic; ev.segd.col0 = (uint32_t)kmin * 256u; ev.segd.ncols = (uint32_t)ncols;
        const uint32_t xstride = (uint32_t)ncols * 2u + 32u;
        ev.xstride_sums = xstride | (sums ? 0x80000000u : 0u);
        ev.mu_off16 = (uint16_t)(xseg_mu_off(B, ncols, sums) / 16u);
        ev.barrier = (uint32_t)s + 1u;   // stage s reads its inputs after barrier s
        if (mix) {
          ev.seg.x = mix_x_off[op] + (uint64_t)kmin * 512u;
          ev.seg.xprev = mix_sums_off[op] + (uint64_t)(kmin * 2) * 3u * nbp * 4u;
          ev.segd.ic = (uint32_t)o.W_desc.ic_pad * 2u;
        } else if (has_mu) {
          const uint8_t* m = static_cast<const uint8_t*>(o.mu_image_dev);
          ev.seg.xprev = (uint64_t)(uintptr_t)o.xprev_fp16_dev;
          ev.seg.mu = (uint64_t)(uintptr_t)(m + RWKVQ_HEADER_BYTES);
          ev.seg.mu_aux = (uint64_t)(uintptr_t)(m + vector_aux_offset(&o.mu_desc));
          ev.segd.mu_bits = (uint16_t)o.mu_desc.bits; ev.segd.mu_entries = (uint16_t)o.mu_desc.entries;
        }
        for (size_t k = i; k <= last; ++k) {
          L[k].u.seg = seg_no;
          L[k].u.ev_index = (uint32_t)(all_events.size() - event_off[c]);
          L[k].u.xcol0 = (uint32_t)(L[k].kt - kmin) * 256u;
          L[k].u.xstride = xstride; L[k].u.gs_off = (uint32_t)B * xstride; L[k].u.nbp = nbp;
        }
        all_events.push_back(ev);
        ++seg_no;
        i = last + 1;
      }
      all_events.push_back(cta_arrivals[c][s + 1]);
    }
    // what each group has to pass between its consecutive segments, and after its last unit of a stage
    uint32_t prev_ev[2] = {0, 0};
    const StepEvent* evs = all_events.data() + event_off[c];
    const uint32_t n_ev = (uint32_t)(all_events.size() - event_off[c]);
    std::vector<uint32_t> arr_idx(n_stages, 0);
    for (uint32_t e = 0; e < n_ev; ++e)
      if (evs[e].kind == EV_ARRIVE && evs[e].barrier > 0u) arr_idx[evs[e].barrier - 1u] = e;
    auto mask_of = [&](uint32_t first, uint32_t last_excl) {
      uint32_t mask = 0;
      for (uint32_t e = first; e < last_excl; ++e)
        if (evs[e].kind == EV_ARRIVE && evs[e].barrier > 0u) mask |= 1u << (e - first);
      return mask;
    };
    for (size_t k = 0; k < n; ++k) {
      const int gidx = (int)(k % kGroups);
      const uint32_t target = L[k].u.ev_index;
      L[k].u.between_mask = (target > prev_ev[gidx] && target - prev_ev[gidx] - 1u <= 32u) ? mask_of(prev_ev[gidx] + 1u, target) : 0u;
      prev_ev[gidx] = target;
      const bool last_of_stage = k + kGroups >= n || L[k + kGroups].stage != L[k].stage;
      const uint32_t arr = arr_idx[L[k].stage];
      if (last_of_stage && arr > target && arr - target <= 32u) {
        L[k].u.after_count = arr - target;
        L[k].u.after_mask = mask_of(target + 1u, arr + 1u);
        prev_ev[gidx] = arr;
      }
    }
    for (size_t k = 0; k < n; ++k) all_units.push_back(L[k].u);
  }
  unit_off[P] = (uint32_t)all_units.size();
  event_off[P] = (uint32_t)all_events.size();

  info->n_units = (uint32_t)all_units.size();
  info->n_events = (uint32_t)all_events.size();
  size_t off = 256;
  info->off_unit_off = off; off += round_up_sz((size_t)(P + 1) * 4, 256);
  info->off_event_off = off; off += round_up_sz((size_t)(P + 1) * 4, 256);
  info->off_units = off; off += round_up_sz(std::max<size_t>(1, all_units.size()) * sizeof(StepUnit), 256);
  info->off_events = off; off += round_up_sz(all_events.size() * sizeof(StepEvent), 256);
  info->off_counter = off; off += round_up_sz((size_t)info->n_barriers * 4, 256);
  info->off_mixops = off; off += round_up_sz(mixops.size() * sizeof(StepMixOp), 256);
  info->off_mixx = off; off += round_up_sz(mixx.size() * sizeof(StepMixX), 256);
  info->off_scratch = off; off += round_up_sz((size_t)scratch_bytes, 256);
  info->total_bytes = off;
  if (out) {
    out->assign(off, 0);
    memcpy(out->data() + info->off_unit_off, unit_off.data(), (size_t)(P + 1) * 4);
    memcpy(out->data() + info->off_event_off, event_off.data(), (size_t)(P + 1) * 4);
    if (!all_units.empty()) memcpy(out->data() + info->off_units, all_units.data(), all_units.size() * sizeof(StepUnit));
    memcpy(out->data() + info->off_events, all_events.data(), all_events.size() * sizeof(StepEvent));
    if (!mixops.empty()) memcpy(out->data() + info->off_mixops, mixops.data(), mixops.size() * sizeof(StepMixOp));
    if (!mixx.empty()) memcpy(out->data() + info->off_mixx, mixx.data(), mixx.size() * sizeof(StepMixX));
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
  for (int i = 0; i < n_ops; ++i) {
    if (i == 0 || ops[i].stage != ops[i - 1].stage) { info.y_lo.push_back(~0ull); info.y_hi.push_back(0ull); }
    const uint64_t lo = (uint64_t)(uintptr_t)ops[i].y_dev, hi = lo + (uint64_t)B * (uint64_t)ops[i].W_desc.oc * 4u;
    info.y_lo.back() = std::min(info.y_lo.back(), lo);
    info.y_hi.back() = std::max(info.y_hi.back(), hi);
  }
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  g_plans[plan_dev] = info;
  return RWKVQ_OK;
}

}  // extern "C"

namespace {
// Inputs that arrive while the step runs (see StepArgs::in_flag), and what the caller needs back to
// order its output copies behind the stage barriers.
struct HostRun {
  const unsigned* in_flag = nullptr;
  unsigned in_base = 0, in_shift = 0;
  uint64_t in_lo = 0, in_hi = 0;
  // out
  unsigned* counter = nullptr;
  unsigned target = 0;
  PlanInfo info;
};

// Every arrival counter that is short of `target` (a run that gave up) is raised to it, so that
// nothing ordered behind a counter waits for ever and the next run starts from a consistent state.
__global__ void step_finish_kernel(unsigned* counter, int n, unsigned target) {
  const int k = (int)(blockIdx.x * blockDim.x + threadIdx.x);
  if (k < n && (int)(counter[k] - target) < 0) counter[k] = target;
}

rwkvq_status step_run_impl(const void* plan_dev, size_t plan_bytes, void* stream, HostRun* hr) {
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
  a.events = reinterpret_cast<const StepEvent*>(p + info.off_events);
  a.unit_off = reinterpret_cast<const uint32_t*>(p + info.off_unit_off);
  a.event_off = reinterpret_cast<const uint32_t*>(p + info.off_event_off);
  a.counter = reinterpret_cast<unsigned*>(const_cast<uint8_t*>(p) + info.off_counter);
  a.status = device_status_ptr();
  if (!a.status) return RWKVQ_ECUDA;
  a.B = info.B; a.n_slots = info.n_slots; a.n_stages = info.n_stages;
  a.mix = info.mix; a.mixops = reinterpret_cast<const StepMixOp*>(p + info.off_mixops);
  a.mixx = reinterpret_cast<const StepMixX*>(p + info.off_mixx);
  a.scratch = const_cast<uint8_t*>(p) + info.off_scratch;
  a.slot_bytes = info.slot_bytes; a.replica_bytes = info.replica_bytes;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  a.target = info.runs * (unsigned)info.P;
  a.poll_limit = info.poll_limit; a.wait_skew = info.wait_skew;
  a.in_flag = nullptr; a.in_base = 0; a.in_shift = 0; a.in_lo = 0; a.in_hi = 0;
  if (hr) {
    a.in_flag = hr->in_flag; a.in_base = hr->in_base; a.in_shift = hr->in_shift; a.in_lo = hr->in_lo; a.in_hi = hr->in_hi;
    hr->counter = a.counter; hr->target = a.target; hr->info = info;
  }
  cudaError_t e = cudaSuccess;
  if (clear_counters) {
    e = cudaMemsetAsync(a.counter, 0, round_up_sz((size_t)info.n_barriers * 4, 256), s);
    if (e != cudaSuccess) return cuda_status(e);
  }
  // batches of 4 and more use the stage pre-pass (StepArgs::mix)
  const void* fn = !info.mix ? (const void*)step_kernel<1, false> : info.NB == 1 ? (const void*)step_kernel<1, true> : (const void*)step_kernel<2, true>;
  e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)info.smem_bytes);
  if (e != cudaSuccess) return cuda_status(e);
  void* params[] = {&a};
  // Cooperative launch: all CTAs must be resident at once because they meet at the stage barrier.
  e = cudaLaunchCooperativeKernel(fn, dim3(info.P), dim3(threads_of(info.NB)), params, info.smem_bytes, s);
  if (e != cudaSuccess) {   // this run will never arrive: have the next one clear the counters
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    auto it = g_plans.find(plan_dev);
    if (it != g_plans.end()) it->second.abort_epoch = abort_epoch() - 1u;
  }
  if (e == cudaSuccess && hr) {
    step_finish_kernel<<<(info.n_barriers + 255u) / 256u, 256, 0, s>>>(a.counter, (int)info.n_barriers, a.target);
    e = cudaGetLastError();
  }
  return cuda_status(e);
}
}  // namespace

extern "C" {

rwkvq_status rwkvq_step_run(const void* plan_dev, size_t plan_bytes, void* stream) {
  return step_run_impl(plan_dev, plan_bytes, stream, nullptr);
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
  const uint32_t* unit_off = reinterpret_cast<const uint32_t*>(image.data() + info.off_unit_off);
  const StepUnit* units = reinterpret_cast<const StepUnit*>(image.data() + info.off_units);
  for (int c = 0; c < n_ctas; ++c) {
    uint32_t items = 0;
    for (uint32_t k = unit_off[c]; k < unit_off[c + 1]; ++k) {
      const StepUnit& u = units[k];
      auto it = op_of_y.find(u.y);
      if (it == op_of_y.end()) return RWKVQ_EINVAL;     // the walk needs distinct output buffers
      const int o = it->second;
      const rwkvq_desc& d = ops[o].W_desc;
      const uint32_t KT = (uint32_t)d.ic_pad / 256u, slices = (uint32_t)d.oc / 16u;
      const uint8_t* payload = static_cast<const uint8_t*>(ops[o].W_image_dev) + RWKVQ_HEADER_BYTES;
      const uint32_t w0 = (u.flags >> 8) & 15u, w1 = (u.flags >> 12) & 15u;
      if (w0 >= w1 || w1 > 8u || u.off0 != w0 * u.rec_bytes) return RWKVQ_EINVAL;
      // the unit's chunks: warp w of the group takes record w of chunk A (and of chunk B, 128 rows below)
      const uint64_t src[2] = {u.src0, u.src1};
      const uint32_t bytes[2] = {u.bytes0, u.bytes1};
      for (int h = 0; h < 2; ++h) {
        if (!bytes[h]) continue;
        if (bytes[h] != (w1 - w0) * u.rec_bytes) return RWKVQ_EINVAL;
        const uint64_t rel = src[h] - (uint64_t)(uintptr_t)payload - (uint64_t)w0 * u.rec_bytes;
        if (rel % u.chunk_bytes) return RWKVQ_EINVAL;
        const uint64_t chunk = rel / u.chunk_bytes;       // mb * KT + kt
        const uint32_t mb = (uint32_t)(chunk / KT), kt = (uint32_t)(chunk % KT);
        if (mb * 128u != u.row0 + 128u * (uint32_t)h) return RWKVQ_EINVAL;
        for (uint32_t w = w0; w < w1; ++w) {
          const uint32_t slice = mb * 8u + w;
          if (slice >= slices) continue;                  // padding rows of the last chunk
          counts_host[base[o] + (size_t)slice * KT + kt] += 1u;
          ++items;
        }
      }
    }
    if (cta_items_host) cta_items_host[c] = items;
  }
  return RWKVQ_OK;
}

}  // extern "C"

namespace {
// Streams, events and the arrival word of host-buffer runs, one set per device.  The stream memory
// operations come from the driver through the runtime's entry-point query (no link to the driver library).
typedef CUresult (*StreamValueFn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
struct HostPipe {
  bool tried = false, ok = false;
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t start = nullptr, h2d_done = nullptr, d2h_done = nullptr;
  unsigned* flag = nullptr;      // device word: chunks arrived so far, over all runs
  unsigned chunks = 0;           // the host's copy of its final value after the last run enqueued
  StreamValueFn wait_value = nullptr, write_value = nullptr;
};
std::mutex g_pipe_mutex;
std::unordered_map<int, HostPipe> g_pipes;
constexpr unsigned kChunkShift = 22;                 // activations arrive in chunks of 4 MB
constexpr size_t kOutGroupBytes = (size_t)2 << 20;   // outputs leave in groups of whole stages of at least 2 MB
constexpr size_t kOverlapMinBytes = (size_t)8 << 20; // steps that copy less run the plain order

HostPipe* host_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  HostPipe& hp = g_pipes[dev];
  if (hp.tried) return hp.ok ? &hp : nullptr;
  hp.tried = true;
  cudaDriverEntryPointQueryResult q1, q2;
  void *f1 = nullptr, *f2 = nullptr;
  if (cudaGetDriverEntryPoint("cuStreamWaitValue32", &f1, cudaEnableDefault, &q1) != cudaSuccess || q1 != cudaDriverEntryPointSuccess || !f1) return nullptr;
  if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &f2, cudaEnableDefault, &q2) != cudaSuccess || q2 != cudaDriverEntryPointSuccess || !f2) return nullptr;
  hp.wait_value = reinterpret_cast<StreamValueFn>(f1);
  hp.write_value = reinterpret_cast<StreamValueFn>(f2);
  if (cudaStreamCreateWithFlags(&hp.h2d, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  if (cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  if (cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) != cudaSuccess) return nullptr;
  if (cudaEventCreateWithFlags(&hp.h2d_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
  if (cudaEventCreateWithFlags(&hp.d2h_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
  if (cudaMalloc(&hp.flag, 256) != cudaSuccess) return nullptr;
  if (cudaMemset(hp.flag, 0, 256) != cudaSuccess) return nullptr;
  // one write and one wait that is already satisfied: if the driver refuses either, stay on the plain path
  if (hp.write_value(hp.h2d, (CUdeviceptr)(uintptr_t)hp.flag, 0u, 0u) != CUDA_SUCCESS) return nullptr;
  if (hp.wait_value(hp.h2d, (CUdeviceptr)(uintptr_t)hp.flag, 0u, CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS) return nullptr;
  if (cudaStreamSynchronize(hp.h2d) != cudaSuccess) return nullptr;
  hp.ok = true;
  return &hp;
}

rwkvq_status run_host_plain(const void* plan_dev, size_t plan_bytes, const void* act_host, void* act_dev, size_t act_bytes,
                            const void* y_dev, void* y_host, size_t y_bytes, void* stream) {
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
}  // namespace

extern "C" {

rwkvq_status rwkvq_step_run_host(const void* plan_dev, size_t plan_bytes, const void* act_host, void* act_dev,
                                 size_t act_bytes, const void* y_dev, void* y_host, size_t y_bytes, void* stream) {
  if ((act_bytes && (!act_host || !act_dev)) || (y_bytes && (!y_dev || !y_host))) return RWKVQ_EINVAL;
  // Small steps: the copies are short and the plain order (copy in, run, copy out on one stream) is best.
  const char* ov = std::getenv("RWKVQ_HOST_OVERLAP");      // "0": always the plain order
  if ((ov && ov[0] == '0') || act_bytes + y_bytes < kOverlapMinBytes)
    return run_host_plain(plan_dev, plan_bytes, act_host, act_dev, act_bytes, y_dev, y_host, y_bytes, stream);
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe* hp = host_pipe();
  if (!hp) return run_host_plain(plan_dev, plan_bytes, act_host, act_dev, act_bytes, y_dev, y_host, y_bytes, stream);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Both side streams start behind everything already enqueued on the caller's stream.
  cudaError_t e = cudaEventRecord(hp->start, s);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hp->h2d, hp->start, 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hp->d2h, hp->start, 0);
  if (e != cudaSuccess) return cuda_status(e);
  // Activations: chunk by chunk on the copy stream; the word counts the chunks that have arrived.
  // They are enqueued BEFORE the launch: streams share a limited number of hardware queues, and a copy
  // enqueued behind the running step in the same queue would start only when the step, which waits for it, ends.
  HostRun hr;
  const size_t chunk = (size_t)1 << kChunkShift;
  const unsigned n_in = (unsigned)((act_bytes + chunk - 1) >> kChunkShift);
  if (n_in) {
    hr.in_flag = hp->flag; hr.in_base = hp->chunks; hr.in_shift = kChunkShift;
    hr.in_lo = (uint64_t)(uintptr_t)act_dev; hr.in_hi = hr.in_lo + act_bytes;
    for (unsigned i = 0; i < n_in; ++i) {
      const size_t off = (size_t)i << kChunkShift, len = std::min(chunk, act_bytes - off);
      e = cudaMemcpyAsync(static_cast<uint8_t*>(act_dev) + off, static_cast<const uint8_t*>(act_host) + off, len, cudaMemcpyHostToDevice, hp->h2d);
      if (e != cudaSuccess) break;
      if (hp->write_value(hp->h2d, (CUdeviceptr)(uintptr_t)hp->flag, hp->chunks + i + 1u, 0u) != CUDA_SUCCESS) { e = cudaErrorUnknown; break; }
    }
    // Whatever happened, the word reaches its final value, so that no stager waits for a chunk in vain.
    if (e != cudaSuccess) hp->write_value(hp->h2d, (CUdeviceptr)(uintptr_t)hp->flag, hp->chunks + n_in, 0u);
    hp->chunks += n_in;
    if (e != cudaSuccess) { cudaStreamSynchronize(hp->h2d); return cuda_status(e); }
  }
  // The step itself, on the caller's stream, at once: its stagers wait for the chunks they read.
  rwkvq_status st = step_run_impl(plan_dev, plan_bytes, stream, &hr);
  if (st != RWKVQ_OK) { cudaStreamSynchronize(hp->h2d); return st; }
  // Outputs: stage by stage behind the stage barriers (the arrival counters of the plan), in groups of
  // whole stages, as long as the stages' outputs lie one behind the other in [y_dev, y_dev + y_bytes).
  if (y_bytes) {
    const PlanInfo& info = hr.info;
    const uint64_t y0 = (uint64_t)(uintptr_t)y_dev, y1 = y0 + y_bytes;
    bool ordered = !info.y_lo.empty();
    uint64_t prev = y0;
    for (size_t k = 0; k < info.y_lo.size() && ordered; ++k) {
      if (info.y_lo[k] < prev || info.y_hi[k] > y1 || info.y_hi[k] < info.y_lo[k]) ordered = false;
      prev = info.y_hi[k];
    }
    const int n_st = info.n_stages;
    size_t done = 0;                               // bytes of the output buffer already handed to copies
    for (int k = 0; k < n_st && e == cudaSuccess; ++k) {
      const bool last = k + 1 == n_st;
      const size_t upto = last || !ordered ? (last ? y_bytes : done) : (size_t)(info.y_hi[k] - y0);
      if (!last && upto - done < kOutGroupBytes) continue;
      if (upto == done) continue;
      // barrier k + 1 closes stage k: every CTA has arrived behind its reductions into these outputs
      if (hp->wait_value(hp->d2h, (CUdeviceptr)(uintptr_t)(hr.counter + (k + 1)), hr.target, CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS) { e = cudaErrorUnknown; break; }
      e = cudaMemcpyAsync(static_cast<uint8_t*>(y_host) + done, static_cast<const uint8_t*>(y_dev) + done, upto - done, cudaMemcpyDeviceToHost, hp->d2h);
      done = upto;
    }
  }
  // The caller's stream ends behind both side streams: synchronizing it covers the whole step.
  if (e == cudaSuccess) e = cudaEventRecord(hp->h2d_done, hp->h2d);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(s, hp->h2d_done, 0);
  if (e == cudaSuccess) e = cudaEventRecord(hp->d2h_done, hp->d2h);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(s, hp->d2h_done, 0);
  return cuda_status(e);
}

}  // extern "C"
