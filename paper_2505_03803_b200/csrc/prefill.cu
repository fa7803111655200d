// Prefill product Y[t][i] = sum_j bf16(w_hat[i][j]) * x_mix[t][j] on the tcgen05 tensor cores.
//
// (1) A pre-pass per product applies the token-shift mix of Appendix A.1 Eq. 20 along the
// sequence (x_mix[t] = X[t] + (X[t-1] - X[t]) (.) mu_hat, X[-1] = xprev0), rounds to bf16 and
// writes the result tile by tile in the shared-memory operand layout of the tensor core (tiles of
// 256 tokens x 64 columns, 128-byte rows, 128-byte swizzle), so that the main kernel fetches an
// operand tile with ONE bulk asynchronous copy.  (2) ONE persistent launch, one CTA per SM, covers
// every product of the call (rwkvq_gemm_prefill_grouped; the single product is a group of one).
// Output tiles of 128 weight rows (one chunk row of the packed image) x 256 tokens are handed out
// by an atomic ticket, longest contraction first, so tiles of different products balance:
//   * a producer thread draws the ticket, publishes the tile to the other roles through a small
//     queue, and streams activation tiles (32 KB per 64 columns, four stages) into shared memory
//     with cp.async.bulk + mbarrier transactions; a second producer thread streams the packed
//     chunks (12-17 KB per 256 columns, as many slots as fit: two to four);
//   * sixteen dequantisation warps in two groups (group g takes the 64-column blocks of parity g,
//     one warp per 16-row record) turn packed codes into bf16, exactly bf16_rne of the fp32
//     rounding of s * (q - z) or of the codebook entry, and store them in the K-major
//     128-byte-swizzled layout, a ring of three tiles; a proxy fence hands them to the tensor core;
//   * one thread issues tcgen05.mma (A = weights 128 x 16, B = activations 256 x 16, fp32
//     accumulators in tensor memory: two stages of 256 columns) and commits to mbarriers;
//   * four epilogue warps read an accumulator stage with tcgen05.ld (lane = weight row, so a warp
//     writes 32 consecutive outputs of one token) while the tensor core fills the other stage
//     with the next tile.
// Every wait is bounded; a wait that gives up raises the device status word and all roles leave
// through the common exit, where tensor memory is freed.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>

#include "../../include/rwkvq.h"
#include "format.h"
#include "host_util.h"
#include "unpack.cuh"

namespace rwkvq {

int* device_status_ptr();  // api_misc.cu

namespace pf {

constexpr int kTileTokens = 256, kTileRows = 128, kKBlock = 64;
constexpr int kXStages = 4, kWStages = 3;   // rings: activation tiles (32 KB); dequantised weight tiles (16 KB)
constexpr uint32_t kXTileBytes = kTileTokens * kKBlock * 2;   // 32 KB: activations of one stage
constexpr uint32_t kWTileBytes = kTileRows * kKBlock * 2;     // 16 KB: dequantised weights of one stage
constexpr int kMaxPackedSlots = 4;                            // packed chunk (+ codebook) slots: as many as fit, at least two
constexpr int kTileQueue = 4;                                 // tiles the producer may run ahead of the slowest role
constexpr uint32_t kCtrlBytes = 1024;
constexpr uint32_t kFixedSmemBytes = kCtrlBytes + kXStages * kXTileBytes + kWStages * kWTileBytes + 1024;  // + alignment slack
constexpr uint32_t kMaxSmemBytes = 232448;                    // per-CTA limit of the architecture
constexpr int kRecordWarps = 8, kDequantGroups = 2, kDequantWarps = kRecordWarps * kDequantGroups, kEpilogueWarps = 4;
constexpr int kThreads = 32 * (3 + kDequantWarps + kEpilogueWarps);   // + activation producer, tensor-core issue, chunk producer
constexpr uint32_t kPollLimit = 1u << 22;
constexpr uint32_t kTmemCols = 512;                           // two accumulator stages of kTileTokens columns
constexpr int kMaxGroup = 16;                                 // products per launch
constexpr size_t kTicketBytes = 256;                          // tail of a product's workspace: the tile ticket

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
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(2000u) : "memory");
  return ok != 0;
}
// Non-blocking test of a phase (1 = complete).  Several tests issued back to back overlap their
// latencies; a blocking try_wait would hold the thread, and with it the tensor-core issue, until
// the phase completes or its time limit passes.
__device__ __forceinline__ uint32_t mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok;
}
// Bounded wait: false after kPollLimit polls (status word set) or once another role has given up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  for (uint32_t it = 0; it < kPollLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicExch(status, (int)RWKVQ_ETIMEOUT);
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// ---- tcgen05 wrappers (one CTA per tile: cta_group::1) ------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* holder_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(holder_smem)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Shared-memory matrix descriptor of a K-major bf16 tile with 128-byte rows and the 128-byte
// swizzle: 8-row groups are 1024 bytes apart; the tile base is 1024-byte aligned and a step of
// 16 columns along K advances the start address by 32 bytes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                            // leading-dimension offset (unused with this swizzle)
  d |= (uint64_t)(1024u >> 4) << 32;                 // stride between 8-row groups
  d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                            // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 32 consecutive columns of an accumulator: register c of lane l = D[lane base + l][col + c].
// The load is asynchronous: the registers hold the data only after tmem_ld_wait on the same array.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
// Waits for every tcgen05.ld of this thread; the array is an in/out operand so that no use of it
// is scheduled before the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
        "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
        "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
        "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
      :: "memory");
}

// Byte offset of element (row r, column k) of a K-major tile with 128-byte rows (64 bf16) and the
// 128-byte swizzle: the 16-byte chunk index is XORed with the row index modulo 8.
__host__ __device__ inline uint32_t sw128_offset(uint32_t r, uint32_t k) {
  return r * 128u + ((((k >> 3) ^ r) & 7u) << 4) + (k & 7u) * 2u;
}

// ---- pre-pass: token-shift mix along the sequence, bf16, operand tile layout -----------------------
__device__ __forceinline__ uint32_t vec_index(const uint8_t* stream, int p, int bits) {
  const uint32_t bitpos = (uint32_t)p * (uint32_t)bits, byte = bitpos >> 3;
  const uint32_t v = (uint32_t)stream[byte] | ((uint32_t)stream[byte + 1] << 8);
  return (v >> (bitpos & 7u)) & ((1u << bits) - 1u);
}

// One block per operand tile (256 tokens x 64 columns).  A thread owns 8 columns (one 16-byte vector)
// and a run of kMixRun consecutive tokens: it decodes its four mu pairs once, reads each row's vector
// once (the previous token's comes from the previous iteration) and writes 16 bytes per token into the
// tile's swizzled rows; the eight threads of a row read and write 128 contiguous bytes.
constexpr int kMixRun = 8;
static_assert(kTileTokens == 32 * kMixRun, "a block of 256 threads covers one tile");
struct MixProduct {
  const __nv_bfloat16* X;
  const __nv_bfloat16* xprev0;
  const uint8_t* mu;
  const uint8_t* mu_aux;
  uint8_t* tiles;
  int mu_bits, ic, KB;
};

struct MixArgs {
  MixProduct p[kMaxGroup];
  unsigned block_start[kMaxGroup + 1];   // first block of each product; [n] = grid size
  int n, M, MT;
};

// One launch mixes the operands of every product of the group: block -> (product, token tile, column block).
__global__ void __launch_bounds__(256) prefill_mix_kernel(const __grid_constant__ MixArgs ma) {
  int pi = 0;
  while (pi + 1 < ma.n && blockIdx.x >= ma.block_start[pi + 1]) ++pi;
  const MixProduct& mp = ma.p[pi];
  const __nv_bfloat16* X = mp.X;
  const __nv_bfloat16* xprev0 = mp.xprev0;
  const uint8_t* mu = mp.mu;
  const uint8_t* mu_aux = mp.mu_aux;
  uint8_t* tiles = mp.tiles;
  const int mu_bits = mp.mu_bits, ic = mp.ic, KB = mp.KB, M = ma.M, MT = ma.MT;
  const unsigned blk = blockIdx.x - ma.block_start[pi];
  const int kb = (int)(blk % (unsigned)KB), mt = (int)(blk / (unsigned)KB);
  if (mt >= MT) return;
  const int cx = threadIdx.x & 7, ty = threadIdx.x >> 3;
  const int c = kb * kKBlock + cx * 8, r0 = ty * kMixRun, t0 = mt * kTileTokens + r0;
  uint8_t* tile = tiles + ((size_t)mt * KB + kb) * kXTileBytes;
  const bool col_ok = c < ic;
  uint4 xr[kMixRun + 1];     // [0] = the token before the run
#pragma unroll
  for (int i = 0; i <= kMixRun; ++i) {
    const int t = t0 + i - 1;
    xr[i] = make_uint4(0u, 0u, 0u, 0u);
    if (col_ok && t < M && (i > 0 || mu != nullptr)) {
      if (t >= 0) xr[i] = *reinterpret_cast<const uint4*>(X + (size_t)t * ic + c);
      else if (xprev0) xr[i] = *reinterpret_cast<const uint4*>(xprev0 + c);
    }
  }
  float2 mf[4];
  if (mu && col_ok) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t mw = reinterpret_cast<const uint32_t*>(mu_aux)[vec_index(mu, (c >> 1) + k, mu_bits)];
      mf[k] = __half22float2(*reinterpret_cast<const __half2*>(&mw));
    }
  }
#pragma unroll
  for (int i = 1; i <= kMixRun; ++i) {
    const int t = t0 + i - 1;
    uint4 out = make_uint4(0u, 0u, 0u, 0u);
    if (col_ok && t < M) {
      out = xr[i];
      if (mu) {
        const uint32_t xs[4] = {xr[i].x, xr[i].y, xr[i].z, xr[i].w}, ps[4] = {xr[i - 1].x, xr[i - 1].y, xr[i - 1].z, xr[i - 1].w};
        uint32_t os[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 xf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&xs[k]));
          const float2 pf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&ps[k]));
          const __nv_bfloat162 o = __floats2bfloat162_rn(fmaf(pf.x - xf.x, mf[k].x, xf.x), fmaf(pf.y - xf.y, mf[k].y, xf.y));
          os[k] = *reinterpret_cast<const uint32_t*>(&o);
        }
        out = make_uint4(os[0], os[1], os[2], os[3]);
      }
    }
    *reinterpret_cast<uint4*>(tile + sw128_offset((uint32_t)(r0 + i - 1), (uint32_t)(cx * 8))) = out;
  }
}

struct PrefillArgs {          // one product of the group
  const uint8_t* payload;   // chunks of the packed image
  const uint8_t* aux;       // VQ codebooks
  const uint8_t* xtiles;    // x_mix in operand tile layout: [MT][KB] tiles of 32 KB
  void* Y;
  int oc, ic, KT, KB, MB, fmt;
  uint32_t chunk_bytes, rec_bytes, cb_bytes;
};

struct GroupArgs {
  PrefillArgs p[kMaxGroup];          // longest contraction first
  int tile_start[kMaxGroup + 1];     // tickets of product i: tile_start[i] .. tile_start[i + 1] - 1
  int n, M, MT, y_dtype;
  int n_slots;                       // packed chunk slots in use (2 .. kMaxPackedSlots)
  uint32_t slot_bytes;               // bytes per slot: the largest chunk + codebook of the group, 128-byte multiple
  unsigned* ticket;                  // cleared before the launch
  int* status;
};

enum { PF_SQ3 = 0, PF_VQ6 = 1, PF_VQ8 = 2 };

struct Ctrl {
  uint64_t cfull[kMaxPackedSlots], cempty[kMaxPackedSlots];
  uint64_t xfull[kXStages], xempty[kXStages], wready[kWStages], wfree[kWStages];
  uint64_t accfull[2], accempty[2];
  uint64_t tqfull[kTileQueue], tqempty[kTileQueue];
  int tileq[kTileQueue];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block");

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// 64 columns (one triple) of an SQ record -> bf16 rows of the weight tile.  `r` are the sixteen
// extracted half2 registers (each half = q + bias exactly).  s * q - s * z with one rounding
// (s * z is exact in fp32: two 11-bit significands) is the fp32 rounding of the exact decode
// s * (q - z); the tile holds its bf16 rounding.
__device__ __forceinline__ void sq_store_triple(const uint32_t (&r)[16], uint32_t sz_lo, uint32_t sz_hi, uint8_t* wtile,
                                                int row_base, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));   // (s, z) of row g
  const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));   // (s, z) of row g + 8
  const float nsz0 = -__fmul_rn(s0.x, s0.y), nsz1 = -__fmul_rn(s1.x, s1.y);
  uint8_t* row0 = wtile + (uint32_t)(row_base + g) * 128u + 8u * (uint32_t)(t & 1);
  const uint32_t sw = (uint32_t)g, c0 = (uint32_t)(t >> 1);     // (row_base + g) % 8 == g: row_base is a multiple of 16
#pragma unroll
  for (int m = 0; m < 4; ++m) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float s = h ? s1.x : s0.x, nsz = h ? nsz1 : nsz0;
      uint32_t out[2];
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const int e = 4 * m + 2 * p + h;
        // (q + bias) - bias is exact in fp16: both are integers below 2048
        const __half2 bias2 = __float2half2_rn((float)(1024 >> rwkvq_sq_pos(e)));
        const float2 qf = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&r[e]), bias2));
        out[p] = pack_bf16(__fmaf_rn(s, qf.x, nsz), __fmaf_rn(s, qf.y, nsz));
      }
      // element (row, 16 m + 4 t): 16-byte chunk (2 m + t / 2) ^ (row % 8), bytes 8 (t % 2) of it; rows g and g + 8 swizzle alike
      const uint32_t off = (uint32_t)h * 1024u + ((((uint32_t)(2 * m) + c0) ^ sw) << 4);
      *reinterpret_cast<uint2*>(row0 + off) = make_uint2(out[0], out[1]);
    }
  }
}

template <int BITS>
__device__ __forceinline__ void vq_store_block(const uint32_t (&w)[2 * BITS], int q, const uint32_t* cb, uint8_t* wtile,
                                               int row_base, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int m = 0; m < 4; ++m) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t out[2];
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        // register R = 2p + h of step j = 4q + m; q is one of four compile-time cases below
        uint32_t idx = 0;
        switch (q) {
          case 0: idx = vq_index<BITS, 2 * BITS>(w, 4 * (0 + m) + 2 * p + h); break;
          case 1: idx = vq_index<BITS, 2 * BITS>(w, 4 * (4 + m) + 2 * p + h); break;
          case 2: idx = vq_index<BITS, 2 * BITS>(w, 4 * (8 + m) + 2 * p + h); break;
          default: idx = vq_index<BITS, 2 * BITS>(w, 4 * (12 + m) + 2 * p + h); break;
        }
        const uint32_t e = cb[idx];
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&e));
        out[p] = pack_bf16(f.x, f.y);
      }
      const uint32_t off = sw128_offset((uint32_t)(row_base + g + 8 * h), (uint32_t)(16 * m + 4 * t));
      *reinterpret_cast<uint2*>(wtile + off) = make_uint2(out[0], out[1]);
    }
  }
}

// Ticket -> product index.  The tile within the product is ticket - tile_start[product], token tile
// major (chunk row = tile % MB, token tile = tile / MB): CTAs that run at the same time read the
// same few activation tiles from L2.
__device__ __forceinline__ int product_of(const GroupArgs& ga, int ticket) {
  int p = 0;
  while (p + 1 < ga.n && ticket >= ga.tile_start[p + 1]) ++p;
  return p;
}

// The next tile of this CTA as published by the producer (-1: none left, or another role gave up).
// Called by whole warps (every lane reads the entry, lane 0 frees it) or by one thread alone.
__device__ __forceinline__ int next_tile(Ctrl* ctrl, uint32_t& tq, bool whole_warp, int lane, volatile int* abortp, int* status) {
  const int slot = (int)(tq % kTileQueue);
  bool ok = mbar_wait(&ctrl->tqfull[slot], (tq / kTileQueue) & 1u, abortp, status);
  if (whole_warp) ok = __all_sync(0xFFFFFFFFu, ok);
  int g = -1;
  if (ok) g = *reinterpret_cast<volatile int*>(&ctrl->tileq[slot]);
  if (whole_warp) __syncwarp();
  if (ok && (!whole_warp || lane == 0)) mbar_arrive(&ctrl->tqempty[slot]);
  ++tq;
  return g;
}

// The blocks of parity DG of one 256-column chunk: registers -> bf16 tiles of the weight ring.
template <int DG>
__device__ __forceinline__ bool dequant_chunk(const uint32_t (&w)[16], const uint4 sz, const uint32_t* cb, int fmt, uint32_t kb0,
                                              Ctrl* ctrl, uint8_t* wring, int dw, int lane, volatile int* abortp, int* status) {
#pragma unroll
  for (int qq = 0; qq < 2; ++qq) {
    const int q = 2 * qq + DG;
    const uint32_t kb = kb0 + (uint32_t)q;
    const int st = (int)(kb % kWStages);
    if (!__all_sync(0xFFFFFFFFu, mbar_wait(&ctrl->wfree[st], ((kb / kWStages) & 1u) ^ 1u, abortp, status))) return false;
    uint8_t* wtile = wring + (size_t)st * kWTileBytes;
    if (fmt == PF_SQ3) {
      uint32_t r[16];
      sq_unpack_triple(w[3 * q], w[3 * q + 1], w[3 * q + 2], r);
      sq_store_triple(r, q < 2 ? sz.x : sz.y, q < 2 ? sz.z : sz.w, wtile, dw * 16, lane);
    } else if (fmt == PF_VQ6) {
      const uint32_t (&w6)[12] = *reinterpret_cast<const uint32_t (*)[12]>(&w[0]);
      vq_store_block<6>(w6, q, cb, wtile, dw * 16, lane);
    } else {
      vq_store_block<8>(w, q, cb, wtile, dw * 16, lane);
    }
    // generic-proxy stores -> visible to the tensor core (async proxy)
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) mbar_arrive(&ctrl->wready[st]);
  }
  return true;
}

__global__ void __launch_bounds__(kThreads, 1) prefill_kernel(const __grid_constant__ GroupArgs ga) {
  extern __shared__ uint8_t smem_raw[];
  // operand tiles need 1024-byte alignment (8 rows of 128 bytes per swizzle group)
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem);
  uint8_t* xring = smem + kCtrlBytes;                        // [kXStages] activation tiles
  uint8_t* wring = xring + kXStages * kXTileBytes;           // [kWStages] dequantised weight tiles
  uint8_t* packed = wring + kWStages * kWTileBytes;          // [n_slots] chunk | codebook
  const uint32_t n_slots = (uint32_t)ga.n_slots, slot_bytes = ga.slot_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abortp = &ctrl->abort_flag;
  const int total = ga.tile_start[ga.n];
  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxPackedSlots; ++s) { mbar_init(&ctrl->cfull[s], 1); mbar_init(&ctrl->cempty[s], kDequantWarps); }
    for (int s = 0; s < kXStages; ++s) { mbar_init(&ctrl->xfull[s], 1); mbar_init(&ctrl->xempty[s], 1); }
    for (int s = 0; s < kWStages; ++s) { mbar_init(&ctrl->wready[s], kRecordWarps); mbar_init(&ctrl->wfree[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&ctrl->accfull[s], 1); mbar_init(&ctrl->accempty[s], kEpilogueWarps); }
    for (int s = 0; s < kTileQueue; ++s) { mbar_init(&ctrl->tqfull[s], 1); mbar_init(&ctrl->tqempty[s], 2 + kDequantWarps + kEpilogueWarps); }
    ctrl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&ctrl->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  if (warp == 0) {
    // ---- activation producer: draws the tickets and streams the activation tiles ---------------------
    if (lane == 0) {
      uint32_t tq = 0, kb_iter = 0;
      bool ok = true;
      while (ok) {
        const int slot = (int)(tq % kTileQueue);
        ok = mbar_wait(&ctrl->tqempty[slot], ((tq / kTileQueue) & 1u) ^ 1u, abortp, ga.status);
        if (!ok) break;
        int g = (int)atomicAdd(ga.ticket, 1u);
        if (g >= total) g = -1;
        *reinterpret_cast<volatile int*>(&ctrl->tileq[slot]) = g;
        mbar_arrive(&ctrl->tqfull[slot]);        // release: the entry is visible to whoever sees the phase complete
        ++tq;
        if (g < 0) break;
        const int pi = product_of(ga, g);
        const PrefillArgs& a = ga.p[pi];
        const int mt = (g - ga.tile_start[pi]) / a.MB, KB = a.KB;
        const uint8_t* src = a.xtiles + (size_t)mt * KB * kXTileBytes;
        for (int kb = 0; kb < KB && ok; ++kb, ++kb_iter) {
          const int st = (int)(kb_iter % kXStages);
          ok = mbar_wait(&ctrl->xempty[st], ((kb_iter / kXStages) & 1u) ^ 1u, abortp, ga.status);
          if (!ok) break;
          mbar_arrive_expect_tx(&ctrl->xfull[st], kXTileBytes);
          bulk_g2s(xring + (size_t)st * kXTileBytes, src + (size_t)kb * kXTileBytes, kXTileBytes, &ctrl->xfull[st]);
        }
      }
      // do not leave while copies issued by this thread may still be landing
      for (uint32_t i = (kb_iter > kXStages ? kb_iter - kXStages : 0); i < kb_iter; ++i)
        for (uint32_t it = 0; it < kPollLimit; ++it) if (mbar_try_wait(&ctrl->xfull[i % kXStages], (i / kXStages) & 1u)) break;
    }
  } else if (warp == 2 + kDequantWarps + kEpilogueWarps) {
    // ---- chunk producer: streams the packed chunks (and codebooks) as far ahead as the slots allow ----
    if (lane == 0) {
      uint32_t tq = 0, ck = 0;
      bool ok = true;
      while (ok) {
        const int g = next_tile(ctrl, tq, false, 0, abortp, ga.status);
        if (g < 0) break;
        const int pi = product_of(ga, g);
        const PrefillArgs& a = ga.p[pi];
        const int cr = (g - ga.tile_start[pi]) % a.MB;
        for (int kt = 0; kt < a.KT && ok; ++kt, ++ck) {
          const uint32_t c = ck % n_slots;
          ok = mbar_wait(&ctrl->cempty[c], ((ck / n_slots) & 1u) ^ 1u, abortp, ga.status);
          if (!ok) break;
          uint8_t* slot_base = packed + (size_t)c * slot_bytes;
          mbar_arrive_expect_tx(&ctrl->cfull[c], a.chunk_bytes + a.cb_bytes);
          bulk_g2s(slot_base, a.payload + (size_t)(cr * a.KT + kt) * a.chunk_bytes, a.chunk_bytes, &ctrl->cfull[c]);
          if (a.cb_bytes) bulk_g2s(slot_base + a.chunk_bytes, a.aux + (size_t)((cr >> 1) * a.KT + kt) * a.cb_bytes, a.cb_bytes, &ctrl->cfull[c]);
        }
      }
      for (uint32_t i = (ck > n_slots ? ck - n_slots : 0); i < ck; ++i)
        for (uint32_t it = 0; it < kPollLimit; ++it) if (mbar_try_wait(&ctrl->cfull[i % n_slots], (i / n_slots) & 1u)) break;
    }
  } else if (warp == 1) {
    // ---- tensor-core issue -----------------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(kTileRows, kTileTokens);
      uint32_t tq = 0, kb_iter = 0, tile_iter = 0;
      bool ok = true;
      while (ok) {
        const int g = next_tile(ctrl, tq, false, 0, abortp, ga.status);
        if (g < 0) break;
        const int KB = ga.p[product_of(ga, g)].KB;
        const uint32_t as = tile_iter & 1u;
        ok = mbar_wait(&ctrl->accempty[as], ((tile_iter >> 1) & 1u) ^ 1u, abortp, ga.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem_base + as * (uint32_t)kTileTokens;
        // The operands of a block are ready when its activation stage has landed and its weight
        // stage has been written.  The two phases are tested together, and those of the next block
        // are tested before this block's instructions are issued, so that the tests' latencies
        // overlap each other and the issue: tested one after the other with blocking waits, the
        // waits and the six instructions of a block took longer than the tensor core needs for it.
        bool ready = false;
        for (int kb = 0; kb < KB && ok; ++kb, ++kb_iter) {
          const int xst = (int)(kb_iter % kXStages), wst = (int)(kb_iter % kWStages);
          const uint32_t xph = (kb_iter / kXStages) & 1u, wph = (kb_iter / kWStages) & 1u;
          for (uint32_t it = 0; !ready; ++it) {
            const uint32_t r0 = mbar_test(&ctrl->xfull[xst], xph);
            const uint32_t r1 = mbar_test(&ctrl->wready[wst], wph);
            ready = (r0 & r1) != 0u;
            if (ready) break;
            if ((it & 63u) == 63u && *abortp) { ok = false; break; }
            if (it >= kPollLimit) {
              *abortp = 1;
              atomicExch(ga.status, (int)RWKVQ_ETIMEOUT);
              ok = false;
              break;
            }
          }
          if (!ok) break;
          tc_fence_after();
          uint32_t n0 = 0u, n1 = 0u;
          if (kb + 1 < KB) {
            const uint32_t nk = kb_iter + 1u;
            n0 = mbar_test(&ctrl->xfull[nk % kXStages], (nk / kXStages) & 1u);
            n1 = mbar_test(&ctrl->wready[nk % kWStages], (nk / kWStages) & 1u);
          }
          const uint32_t xs = smem_u32(xring + (size_t)xst * kXTileBytes);
          const uint32_t wa = smem_u32(wring + (size_t)wst * kWTileBytes);
#pragma unroll
          for (int k = 0; k < kKBlock / 16; ++k)
            umma_bf16(acc, smem_desc_sw128(wa + k * 32), smem_desc_sw128(xs + k * 32), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(&ctrl->wfree[wst]);
          umma_commit(&ctrl->xempty[xst]);
          ready = (n0 & n1) != 0u;
        }
        if (ok) umma_commit(&ctrl->accfull[as]);
        ++tile_iter;
      }
    }
  } else if (warp < 2 + kDequantWarps) {
    // ---- dequantisation: warp dw takes record dw (16 rows) of the chunk, group dg the blocks of parity dg ----
    const int dw = (warp - 2) & 7, dg = (warp - 2) >> 3, g8 = lane >> 2;
    uint32_t tq = 0, ck = 0, kb0 = 0;      // kb0: 64-column blocks before the current chunk
    bool ok = true;
    while (ok) {
      const int g = next_tile(ctrl, tq, true, lane, abortp, ga.status);
      if (g < 0) break;
      const PrefillArgs& a = ga.p[product_of(ga, g)];
      const int fmt = a.fmt, KT = a.KT;
      const uint32_t chunk_bytes = a.chunk_bytes, rec_bytes = a.rec_bytes;
      for (int kt = 0; kt < KT && ok; ++kt, ++ck, kb0 += 4) {
        const uint32_t c = ck % n_slots;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(&ctrl->cfull[c], (ck / n_slots) & 1u, abortp, ga.status));
        if (!ok) break;
        const uint8_t* slot_base = packed + (size_t)c * slot_bytes;
        const uint8_t* rec = slot_base + (size_t)dw * rec_bytes;
        const uint32_t* cb = reinterpret_cast<const uint32_t*>(slot_base + chunk_bytes);
        uint32_t w[16];
        uint4 sz = make_uint4(0, 0, 0, 0);
        const int nplanes = fmt == PF_VQ8 ? 4 : 3;
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (p < nplanes) v = *reinterpret_cast<const uint4*>(rec + p * 512 + lane * 16);
          w[4 * p] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
        }
        if (fmt == PF_SQ3) sz = *reinterpret_cast<const uint4*>(rec + RWKVQ_SQ_CODE_BYTES + g8 * 16);
        // SQ needs nothing more from the packed slot (the codes are in registers): free it now.
        // VQ still reads the codebook while it expands the blocks.
        const bool early = fmt == PF_SQ3;
        __syncwarp();
        if (early && lane == 0) mbar_arrive(&ctrl->cempty[c]);
        ok = dg == 0 ? dequant_chunk<0>(w, sz, cb, fmt, kb0, ctrl, wring, dw, lane, abortp, ga.status)
                     : dequant_chunk<1>(w, sz, cb, fmt, kb0, ctrl, wring, dw, lane, abortp, ga.status);
        __syncwarp();
        if (!early && ok && lane == 0) mbar_arrive(&ctrl->cempty[c]);
      }
    }
  } else if (warp < 2 + kDequantWarps + kEpilogueWarps) {
    // ---- epilogue: warp quarter qd reads lanes 32 qd .. 32 qd + 31 (weight rows) of an accumulator stage ----
    const int qd = warp & 3;
    uint32_t tq = 0, tile_iter = 0;
    bool ok = true;
    while (ok) {
      const int g = next_tile(ctrl, tq, true, lane, abortp, ga.status);
      if (g < 0) break;
      const int pi = product_of(ga, g);
      const PrefillArgs& a = ga.p[pi];
      const int local = g - ga.tile_start[pi], cr = local % a.MB, mt = local / a.MB;
      const uint32_t as = tile_iter & 1u;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(&ctrl->accfull[as], (tile_iter >> 1) & 1u, abortp, ga.status));
      if (!ok) break;
      tc_fence_after();
      const int t0 = mt * kTileTokens, row = cr * kTileRows + qd * 32 + lane, oc = a.oc;
      const uint32_t acc = tmem_base + as * (uint32_t)kTileTokens + ((uint32_t)(qd * 32) << 16);
      const bool row_ok = row < oc;
      float* yf = static_cast<float*>(a.Y) + row;
      __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(a.Y) + row;
      const bool f32 = ga.y_dtype == RWKVQ_F32;
      // two register buffers: the load of the next 32 columns is in flight while these are stored
      uint32_t ra[32], rb[32];
      tmem_ld32_issue(acc, ra);
#pragma unroll 1
      for (int cc = 0; cc < kTileTokens / 32; cc += 2) {
        tmem_ld_wait(ra);
        tmem_ld32_issue(acc + (uint32_t)((cc + 1) * 32), rb);
        if (row_ok) {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const int t = t0 + cc * 32 + c;
            if (t < ga.M) {
              if (f32) yf[(size_t)t * oc] = __uint_as_float(ra[c]);
              else yb[(size_t)t * oc] = __float2bfloat16_rn(__uint_as_float(ra[c]));
            }
          }
        }
        tmem_ld_wait(rb);
        if (cc + 2 < kTileTokens / 32) tmem_ld32_issue(acc + (uint32_t)((cc + 2) * 32), ra);
        if (row_ok) {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const int t = t0 + (cc + 1) * 32 + c;
            if (t < ga.M) {
              if (f32) yf[(size_t)t * oc] = __uint_as_float(rb[c]);
              else yb[(size_t)t * oc] = __float2bfloat16_rn(__uint_as_float(rb[c]));
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl->accempty[as]);
      ++tile_iter;
    }
  }
  // common exit: every role's loops are bounded, so all threads arrive here
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace pf
}  // namespace rwkvq

using namespace rwkvq;

namespace {

struct HostProduct {
  pf::PrefillArgs a;
  const void* X; const void* xprev0;
  const uint8_t* mup; const uint8_t* mua; int mu_bits;
  uint8_t* ws;
};

rwkvq_status check_product(const rwkvq_prefill_op& o, int M, HostProduct* out) {
  const rwkvq_desc* d = o.W_desc;
  if (!d || !o.W_image_dev || !o.X_bf16_dev || !o.Y_dev) return RWKVQ_EINVAL;
  if (o.mu_image_dev && !o.mu_desc) return RWKVQ_EINVAL;
  if (!o.mu_image_dev && o.xprev0_bf16_dev) return RWKVQ_EINVAL;
  if (d->oc == 1) return RWKVQ_ESHAPE;
  rwkvq_status st = check_matrix_desc(d);
  if (st != RWKVQ_OK) return st;
  if (o.mu_image_dev) {
    st = check_vector_desc(o.mu_desc, d->ic);
    if (st != RWKVQ_OK) return st;
  }
  if (d->ic % 8) return RWKVQ_ESHAPE;
  if (!aligned16(o.W_image_dev) || !aligned16(o.X_bf16_dev) || !aligned16(o.Y_dev) || (o.mu_image_dev && !aligned16(o.mu_image_dev)) ||
      (o.xprev0_bf16_dev && !aligned16(o.xprev0_bf16_dev)))
    return RWKVQ_EALIGN;
  const size_t need = rwkvq_prefill_workspace_bytes(d, M, o.mu_image_dev != nullptr);
  if (!o.workspace_dev || o.workspace_bytes < need) return RWKVQ_ENOMEM;
  if ((reinterpret_cast<uintptr_t>(o.workspace_dev) & 127u) != 0) return RWKVQ_EALIGN;
  const uint8_t* img = static_cast<const uint8_t*>(o.W_image_dev);
  pf::PrefillArgs& a = out->a;
  a.payload = img + RWKVQ_HEADER_BYTES;
  a.aux = img + matrix_aux_offset(d);
  a.xtiles = static_cast<const uint8_t*>(o.workspace_dev);
  a.Y = o.Y_dev;
  a.oc = d->oc; a.ic = d->ic;
  a.KT = d->ic_pad / 256; a.KB = a.KT * 4; a.MB = d->oc_pad / 128;
  a.fmt = d->method == RWKVQ_SQ ? pf::PF_SQ3 : (d->bits == 6 ? pf::PF_VQ6 : pf::PF_VQ8);
  a.rec_bytes = d->method == RWKVQ_SQ ? (uint32_t)RWKVQ_SQ_RECORD_BYTES : rwkvq_vq_record_bytes(d->bits);
  a.chunk_bytes = 8u * a.rec_bytes;
  a.cb_bytes = d->method == RWKVQ_SQ ? 0u : (uint32_t)d->entries * 4u;
  out->X = o.X_bf16_dev; out->xprev0 = o.xprev0_bf16_dev;
  out->mup = nullptr; out->mua = nullptr; out->mu_bits = 0;
  if (o.mu_image_dev) {
    const uint8_t* m = static_cast<const uint8_t*>(o.mu_image_dev);
    out->mup = m + RWKVQ_HEADER_BYTES; out->mua = m + vector_aux_offset(o.mu_desc); out->mu_bits = o.mu_desc->bits;
  }
  out->ws = static_cast<uint8_t*>(o.workspace_dev);
  return RWKVQ_OK;
}

}  // namespace

extern "C" {

size_t rwkvq_prefill_workspace_bytes(const rwkvq_desc* d, int M, int has_mu) {
  (void)has_mu;   // the operand tiles are written whether or not a token shift is applied
  if (!d || M <= 0 || check_matrix_desc(d) != RWKVQ_OK) return 0;
  const size_t MT = ((size_t)M + pf::kTileTokens - 1) / pf::kTileTokens, KB = (size_t)d->ic_pad / pf::kKBlock;
  return MT * KB * pf::kXTileBytes + pf::kTicketBytes;
}

rwkvq_status rwkvq_gemm_prefill_grouped(const rwkvq_prefill_op* ops, int n_ops, int M, int y_dtype, void* stream) {
  if (!ops || n_ops <= 0 || M <= 0) return RWKVQ_EINVAL;
  if (n_ops > pf::kMaxGroup) return RWKVQ_EUNSUPPORTED;
  if (y_dtype != RWKVQ_F32 && y_dtype != RWKVQ_BF16) return RWKVQ_EINVAL;
  HostProduct hp[pf::kMaxGroup];
  for (int i = 0; i < n_ops; ++i) {
    const rwkvq_status st = check_product(ops[i], M, &hp[i]);
    if (st != RWKVQ_OK) return st;
    for (int j = 0; j < i; ++j)
      if (ops[j].Y_dev == ops[i].Y_dev || ops[j].workspace_dev == ops[i].workspace_dev) return RWKVQ_EINVAL;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int MT = (M + pf::kTileTokens - 1) / pf::kTileTokens;
  // longest contraction first: the long tiles are dealt before the short ones fill the gaps
  int order[pf::kMaxGroup];
  for (int i = 0; i < n_ops; ++i) order[i] = i;
  std::stable_sort(order, order + n_ops, [&](int x, int y) { return hp[x].a.KB > hp[y].a.KB; });
  pf::GroupArgs ga;
  memset(&ga, 0, sizeof(ga));
  ga.n = n_ops; ga.M = M; ga.MT = MT; ga.y_dtype = y_dtype;
  ga.status = device_status_ptr();
  if (!ga.status) return RWKVQ_ECUDA;
  long long total = 0;
  for (int i = 0; i < n_ops; ++i) {
    ga.p[i] = hp[order[i]].a;
    ga.tile_start[i] = (int)total;
    total += (long long)ga.p[i].MB * MT;
    if (total > 0x3FFFFFFF) return RWKVQ_EUNSUPPORTED;
  }
  ga.tile_start[n_ops] = (int)total;
  uint32_t slot = 0;
  for (int i = 0; i < n_ops; ++i) slot = std::max(slot, (ga.p[i].chunk_bytes + ga.p[i].cb_bytes + 127u) & ~127u);
  ga.slot_bytes = slot;
  ga.n_slots = (int)std::min<uint32_t>(pf::kMaxPackedSlots, (pf::kMaxSmemBytes - pf::kFixedSmemBytes) / slot);
  if (ga.n_slots < 2) return RWKVQ_EUNSUPPORTED;
  const uint32_t smem_bytes = pf::kFixedSmemBytes + (uint32_t)ga.n_slots * slot;
  const HostProduct& first = hp[order[0]];
  ga.ticket = reinterpret_cast<unsigned*>(first.ws + (size_t)MT * first.a.KB * pf::kXTileBytes);
  cudaError_t e = cudaMemsetAsync(ga.ticket, 0, sizeof(unsigned), s);
  if (e != cudaSuccess) return cuda_status(e);
  // pre-pass: the operands of all products in one launch, in the order the tiles will be dealt
  pf::MixArgs ma;
  memset(&ma, 0, sizeof(ma));
  ma.n = n_ops; ma.M = M; ma.MT = MT;
  unsigned long long mix_blocks = 0;
  for (int i = 0; i < n_ops; ++i) {
    const HostProduct& h = hp[order[i]];
    pf::MixProduct& mp = ma.p[i];
    mp.X = static_cast<const __nv_bfloat16*>(h.X); mp.xprev0 = static_cast<const __nv_bfloat16*>(h.xprev0);
    mp.mu = h.mup; mp.mu_aux = h.mua; mp.tiles = h.ws; mp.mu_bits = h.mu_bits; mp.ic = h.a.ic; mp.KB = h.a.KB;
    ma.block_start[i] = (unsigned)mix_blocks;
    mix_blocks += (unsigned long long)MT * (unsigned long long)h.a.KB;
    if (mix_blocks > 0x7FFFFFFFull) return RWKVQ_EUNSUPPORTED;
  }
  ma.block_start[n_ops] = (unsigned)mix_blocks;
  pf::prefill_mix_kernel<<<(unsigned)mix_blocks, 256, 0, s>>>(ma);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_status(e);
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  e = cudaFuncSetAttribute(pf::prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pf::kMaxSmemBytes);
  if (e != cudaSuccess) return cuda_status(e);
  const int grid = total < sms ? (int)total : sms;
  pf::prefill_kernel<<<grid, pf::kThreads, smem_bytes, s>>>(ga);
  return cuda_status(cudaGetLastError());
}

rwkvq_status rwkvq_gemm_prefill(const rwkvq_desc* d, const void* W, const rwkvq_desc* mud, const void* mu, const void* X,
                                const void* xprev0, int M, void* Y, int y_dtype, void* ws, size_t ws_bytes, void* stream) {
  if (!d || !W || !X || !Y || M <= 0) return RWKVQ_EINVAL;
  if (mu && !mud) return RWKVQ_EINVAL;
  rwkvq_prefill_op op;
  op.W_desc = d; op.W_image_dev = W; op.mu_desc = mud; op.mu_image_dev = mu; op.X_bf16_dev = X; op.xprev0_bf16_dev = xprev0;
  op.Y_dev = Y; op.workspace_dev = ws; op.workspace_bytes = ws_bytes;
  return rwkvq_gemm_prefill_grouped(&op, 1, M, y_dtype, stream);
}

}  // extern "C"
