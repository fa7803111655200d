// Prefill product Y[t][i] = sum_j bf16(w_hat[i][j]) * x_mix[t][j] on the tcgen05 tensor cores.
//
// Two launches.  (1) A pre-pass applies the token-shift mix of Appendix A.1 Eq. 20 along the
// sequence (x_mix[t] = X[t] + (X[t-1] - X[t]) (.) mu_hat, X[-1] = xprev0), rounds to bf16 and
// writes the result tile by tile in the shared-memory operand layout of the tensor core (tiles of
// 256 tokens x 64 columns, 128-byte rows, 128-byte swizzle), so that the main kernel fetches an
// operand tile with ONE bulk asynchronous copy.  (2) The main kernel is persistent, one CTA per
// SM, each looping over output tiles of 256 weight rows (two chunks of the packed image) x 256
// tokens, so that one activation tile feeds two products:
//   * a producer warp streams packed chunk pairs (27-34 KB per 256 columns) and activation tiles
//     (32 KB per 64 columns) into shared memory with cp.async.bulk + mbarrier transactions;
//   * sixteen dequantisation warps (one group of eight per row half, one warp per 16-row record)
//     turn packed codes into bf16 with
//     the shared unpack routines, exactly bf16_rne(s * (q - z)) or bf16_rne(codebook entry), and
//     store them in the K-major 128-byte-swizzled layout; a proxy fence hands them to the tensor core;
//   * one thread issues tcgen05.mma (A = weights 128 x 16, B = activations 256 x 16, fp32
//     accumulators in tensor memory, one of 256 columns per row half) and commits to mbarriers;
//   * four epilogue warps read the accumulators with tcgen05.ld (lane = weight row, so a warp
//     writes 32 consecutive outputs of one token) while the next tile's operands stream in.
// Every wait is bounded; a wait that gives up raises the device status word and all roles leave
// through the common exit, where tensor memory is freed.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rwkvq.h"
#include "format.h"
#include "host_util.h"
#include "unpack.cuh"

namespace rwkvq {

int* device_status_ptr();  // api_misc.cu

namespace pf {

constexpr int kTileTokens = 256, kTileRows = 128, kKBlock = 64;
constexpr int kXStages = 3, kWStages = 2;   // rings: activation tiles (32 KB); dequantised weight tiles (16 KB), one ring per row half
constexpr uint32_t kXTileBytes = kTileTokens * kKBlock * 2;   // 32 KB: activations of one stage
constexpr uint32_t kWTileBytes = kTileRows * kKBlock * 2;     // 16 KB: dequantised weights of one stage
constexpr uint32_t kPackedSlot = 2 * 8 * 2048 + 1024;         // two largest chunks (VQ, 8-bit) + their codebook
constexpr int kPackedSlots = 1;
constexpr uint32_t kCtrlBytes = 1024;
constexpr uint32_t kSmemBytes = kCtrlBytes + kXStages * kXTileBytes + 2 * kWStages * kWTileBytes + kPackedSlots * kPackedSlot + 1024;  // + alignment slack
constexpr int kRecordWarps = 8, kDequantGroups = 2, kDequantWarps = kRecordWarps * kDequantGroups, kEpilogueWarps = 4;
constexpr int kThreads = 32 * (2 + kDequantWarps + kEpilogueWarps);
constexpr uint32_t kPollLimit = 1u << 22;
constexpr uint32_t kTmemCols = 512;

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
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
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

// One thread per 8 consecutive columns of one (padded) token row.
__global__ void __launch_bounds__(256) prefill_mix_kernel(const __nv_bfloat16* X, const __nv_bfloat16* xprev0, const uint8_t* mu,
                                                          const uint8_t* mu_aux, int mu_bits, int M, int ic, int KB, int MT,
                                                          uint8_t* tiles) {
  const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int vec_per_row = KB * 8;
  if (v >= (long long)MT * kTileTokens * vec_per_row) return;
  const int t = (int)(v / vec_per_row), c = (int)(v % vec_per_row) * 8;
  uint4 out = make_uint4(0u, 0u, 0u, 0u);
  if (t < M && c < ic) {
    const uint4 xr = *reinterpret_cast<const uint4*>(X + (size_t)t * ic + c);
    out = xr;
    if (mu) {
      uint4 pr = make_uint4(0u, 0u, 0u, 0u);
      if (t > 0) pr = *reinterpret_cast<const uint4*>(X + (size_t)(t - 1) * ic + c);
      else if (xprev0) pr = *reinterpret_cast<const uint4*>(xprev0 + c);
      const uint32_t xs[4] = {xr.x, xr.y, xr.z, xr.w}, ps[4] = {pr.x, pr.y, pr.z, pr.w};
      uint32_t os[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t mw = reinterpret_cast<const uint32_t*>(mu_aux)[vec_index(mu, (c >> 1) + k, mu_bits)];
        const float2 mf = __half22float2(*reinterpret_cast<const __half2*>(&mw));
        const float2 xf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&xs[k]));
        const float2 pf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&ps[k]));
        const __nv_bfloat162 o = __floats2bfloat162_rn(fmaf(pf.x - xf.x, mf.x, xf.x), fmaf(pf.y - xf.y, mf.y, xf.y));
        os[k] = *reinterpret_cast<const uint32_t*>(&o);
      }
      out = make_uint4(os[0], os[1], os[2], os[3]);
    }
  }
  const int mt = t / kTileTokens, r = t % kTileTokens, kb = c / kKBlock;
  uint8_t* tile = tiles + ((size_t)mt * KB + kb) * kXTileBytes;
  *reinterpret_cast<uint4*>(tile + sw128_offset((uint32_t)r, (uint32_t)(c % kKBlock))) = out;
}

struct PrefillArgs {
  const uint8_t* payload;   // chunks of the packed image
  const uint8_t* aux;       // VQ codebooks
  const uint8_t* xtiles;    // x_mix in operand tile layout: [MT][KB] tiles of 32 KB
  void* Y;
  int* status;
  int oc, ic, M, KT, KB, MB, MT, n_tiles, fmt, entries, y_dtype;
  uint32_t chunk_bytes, rec_bytes, cb_bytes;
};

enum { PF_SQ3 = 0, PF_VQ6 = 1, PF_VQ8 = 2 };

struct Ctrl {
  uint64_t wfull[kPackedSlots], wempty[kPackedSlots];
  uint64_t xfull[kXStages], xempty[kXStages], wready[2][kWStages], wfree[2][kWStages];
  uint64_t accfull, accempty;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block");

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// 64 columns (one triple) of an SQ record -> bf16 rows of the weight tile.  `r` are the sixteen
// extracted half2 registers (each half = q + bias exactly); every value is
// bf16_rne(fmul_rn(s, fsub_rn(q, z))), the rounding of the exact decode.
__device__ __forceinline__ void sq_store_triple(const uint32_t (&r)[16], uint32_t sz_lo, uint32_t sz_hi, uint8_t* wtile,
                                                int row_base, int lane) {
  const int g = lane >> 2, t = lane & 3;
  const float2 s0 = __half22float2(*reinterpret_cast<const __half2*>(&sz_lo));   // (s, z) of row g
  const float2 s1 = __half22float2(*reinterpret_cast<const __half2*>(&sz_hi));   // (s, z) of row g + 8
#pragma unroll
  for (int m = 0; m < 4; ++m) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float s = h ? s1.x : s0.x, z = h ? s1.y : s0.y;
      uint32_t out[2];
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const int e = 4 * m + 2 * p + h;
        // (q + bias) - bias is exact in fp16: both are integers below 2048
        const __half2 bias2 = __float2half2_rn((float)(1024 >> rwkvq_sq_pos(e)));
        const float2 qf = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&r[e]), bias2));
        const float v0 = __fmul_rn(s, __fsub_rn(qf.x, z));
        const float v1 = __fmul_rn(s, __fsub_rn(qf.y, z));
        out[p] = pack_bf16(v0, v1);
      }
      const uint32_t off = sw128_offset((uint32_t)(row_base + g + 8 * h), (uint32_t)(16 * m + 4 * t));
      *reinterpret_cast<uint2*>(wtile + off) = make_uint2(out[0], out[1]);
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

__global__ void __launch_bounds__(kThreads, 1) prefill_kernel(const PrefillArgs a) {
  extern __shared__ uint8_t smem_raw[];
  // operand tiles need 1024-byte alignment (8 rows of 128 bytes per swizzle group)
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem);
  uint8_t* xring = smem + kCtrlBytes;                        // [kXStages] activation tiles
  uint8_t* wring = xring + kXStages * kXTileBytes;           // [2 row halves][kWStages] dequantised weight tiles
  uint8_t* packed = wring + 2 * kWStages * kWTileBytes;      // [chunk A | chunk B | codebook]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abortp = &ctrl->abort_flag;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kPackedSlots; ++s) { mbar_init(&ctrl->wfull[s], 1); mbar_init(&ctrl->wempty[s], kDequantWarps); }
    for (int s = 0; s < kXStages; ++s) { mbar_init(&ctrl->xfull[s], 1); mbar_init(&ctrl->xempty[s], 1); }
    for (int h = 0; h < 2; ++h)
      for (int s = 0; s < kWStages; ++s) { mbar_init(&ctrl->wready[h][s], kRecordWarps); mbar_init(&ctrl->wfree[h][s], 1); }
    mbar_init(&ctrl->accfull, 1); mbar_init(&ctrl->accempty, kEpilogueWarps);
    ctrl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&ctrl->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;
  // A tile is 256 weight rows (row pair tr: chunks 2 tr and 2 tr + 1 of the image) x 256 tokens: one
  // activation tile feeds two products, which halves the activation traffic from L2 per FLOP.
  // The last row pair of a matrix with an odd number of chunks has only its first half.

  if (warp == 0) {
    // ---- producer ------------------------------------------------------------------------------
    if (lane == 0) {
      uint32_t kt_iter = 0, kb_iter = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < a.n_tiles && ok; tile += gridDim.x) {
        const int tr = tile / a.MT, mt = tile % a.MT;
        const bool has_b = 2 * tr + 1 < a.MB;
        for (int kt = 0; kt < a.KT && ok; ++kt, ++kt_iter) {
          ok = mbar_wait(&ctrl->wempty[0], (kt_iter & 1u) ^ 1u, abortp, a.status);
          if (!ok) break;
          mbar_arrive_expect_tx(&ctrl->wfull[0], a.chunk_bytes * (has_b ? 2u : 1u) + a.cb_bytes);
          bulk_g2s(packed, a.payload + (size_t)((2 * tr) * a.KT + kt) * a.chunk_bytes, a.chunk_bytes, &ctrl->wfull[0]);
          if (has_b) bulk_g2s(packed + a.chunk_bytes, a.payload + (size_t)((2 * tr + 1) * a.KT + kt) * a.chunk_bytes, a.chunk_bytes, &ctrl->wfull[0]);
          if (a.cb_bytes) bulk_g2s(packed + 2 * a.chunk_bytes, a.aux + (size_t)(tr * a.KT + kt) * a.cb_bytes, a.cb_bytes, &ctrl->wfull[0]);
          for (int q = 0; q < 4 && ok; ++q, ++kb_iter) {
            const int st = (int)(kb_iter % kXStages);
            ok = mbar_wait(&ctrl->xempty[st], ((kb_iter / kXStages) & 1u) ^ 1u, abortp, a.status);
            if (!ok) break;
            mbar_arrive_expect_tx(&ctrl->xfull[st], kXTileBytes);
            bulk_g2s(xring + (size_t)st * kXTileBytes, a.xtiles + ((size_t)mt * a.KB + (kt * 4 + q)) * kXTileBytes, kXTileBytes, &ctrl->xfull[st]);
          }
        }
      }
      // do not leave while copies issued by this thread may still be landing
      for (uint32_t i = (kb_iter > kXStages ? kb_iter - kXStages : 0); i < kb_iter; ++i)
        for (uint32_t it = 0; it < kPollLimit; ++it) if (mbar_try_wait(&ctrl->xfull[i % kXStages], (i / kXStages) & 1u)) break;
      if (kt_iter > 0)
        for (uint32_t it = 0; it < kPollLimit; ++it) if (mbar_try_wait(&ctrl->wfull[0], (kt_iter - 1u) & 1u)) break;
    }
  } else if (warp == 1) {
    // ---- tensor-core issue -----------------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(kTileRows, kTileTokens);
      uint32_t kb_iter = 0, kb_b = 0, tile_iter = 0;     // kb_b counts the blocks of tiles that have a second half
      bool ok = true;
      for (int tile = blockIdx.x; tile < a.n_tiles && ok; tile += gridDim.x, ++tile_iter) {
        const int tr = tile / a.MT;
        const bool has_b = 2 * tr + 1 < a.MB;
        ok = mbar_wait(&ctrl->accempty, (tile_iter & 1u) ^ 1u, abortp, a.status);
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < a.KB && ok; ++kb, ++kb_iter) {
          const int xst = (int)(kb_iter % kXStages), sa = (int)(kb_iter % kWStages);
          ok = mbar_wait(&ctrl->xfull[xst], (kb_iter / kXStages) & 1u, abortp, a.status) &&
               mbar_wait(&ctrl->wready[0][sa], (kb_iter / kWStages) & 1u, abortp, a.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t xs = smem_u32(xring + (size_t)xst * kXTileBytes);
          const uint32_t wa = smem_u32(wring + (size_t)sa * kWTileBytes);
#pragma unroll
          for (int k = 0; k < kKBlock / 16; ++k)
            umma_bf16(tmem_base, smem_desc_sw128(wa + k * 32), smem_desc_sw128(xs + k * 32), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(&ctrl->wfree[0][sa]);
          if (has_b) {
            const int sb = (int)(kb_b % kWStages);
            ok = mbar_wait(&ctrl->wready[1][sb], (kb_b / kWStages) & 1u, abortp, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t wb = smem_u32(wring + (size_t)(kWStages + sb) * kWTileBytes);
#pragma unroll
            for (int k = 0; k < kKBlock / 16; ++k)
              umma_bf16(tmem_base + (uint32_t)kTileTokens, smem_desc_sw128(wb + k * 32), smem_desc_sw128(xs + k * 32), idesc, (kb > 0 || k > 0) ? 1u : 0u);
            umma_commit(&ctrl->wfree[1][sb]);
            ++kb_b;
          }
          umma_commit(&ctrl->xempty[xst]);    // the activation tile is free once both products have read it
        }
        if (ok) umma_commit(&ctrl->accfull);
      }
    }
  } else if (warp < 2 + kDequantWarps) {
    // ---- dequantisation: group dg takes row half dg of the tile, warp dw its record dw (16 rows) ----
    const int dw = (warp - 2) & 7, dg = (warp - 2) >> 3, g = lane >> 2;
    uint32_t kt_iter = 0, kbm = 0;      // kbm: 64-column blocks this group has produced
    bool ok = true;
    for (int tile = blockIdx.x; tile < a.n_tiles && ok; tile += gridDim.x) {
      const int tr = tile / a.MT;
      const bool mine = dg == 0 || 2 * tr + 1 < a.MB;     // the second half may be absent
      for (int kt = 0; kt < a.KT && ok; ++kt, ++kt_iter) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(&ctrl->wfull[0], kt_iter & 1u, abortp, a.status));
        if (!ok) break;
        const uint8_t* rec = packed + (size_t)dg * a.chunk_bytes + (size_t)dw * a.rec_bytes;
        const uint32_t* cb = reinterpret_cast<const uint32_t*>(packed + 2 * a.chunk_bytes);
        uint32_t w[16];
        uint4 sz = make_uint4(0, 0, 0, 0);
        const int nplanes = a.fmt == PF_VQ8 ? 4 : 3;
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (mine && p < nplanes) v = *reinterpret_cast<const uint4*>(rec + p * 512 + lane * 16);
          w[4 * p] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
        }
        if (mine && a.fmt == PF_SQ3) sz = *reinterpret_cast<const uint4*>(rec + RWKVQ_SQ_CODE_BYTES + g * 16);
        // SQ needs nothing more from the packed slot (the codes are in registers): free it now so
        // that the next 256 columns stream in while these are expanded.  VQ still reads the codebook.
        const bool early = a.fmt == PF_SQ3;
        __syncwarp();
        if (early && lane == 0) mbar_arrive(&ctrl->wempty[0]);
        if (mine) {
#pragma unroll
          for (int q = 0; q < 4; ++q, ++kbm) {
            const int st = (int)(kbm % kWStages);
            if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(&ctrl->wfree[dg][st], ((kbm / kWStages) & 1u) ^ 1u, abortp, a.status));
            if (ok) {
              uint8_t* wtile = wring + (size_t)(dg * kWStages + st) * kWTileBytes;
              if (a.fmt == PF_SQ3) {
                uint32_t r[16];
                sq_unpack_triple(w[3 * q], w[3 * q + 1], w[3 * q + 2], r);
                sq_store_triple(r, q < 2 ? sz.x : sz.y, q < 2 ? sz.z : sz.w, wtile, dw * 16, lane);
              } else if (a.fmt == PF_VQ6) {
                const uint32_t (&w6)[12] = *reinterpret_cast<const uint32_t (*)[12]>(&w[0]);
                vq_store_block<6>(w6, q, cb, wtile, dw * 16, lane);
              } else {
                vq_store_block<8>(w, q, cb, wtile, dw * 16, lane);
              }
              // generic-proxy stores -> visible to the tensor core (async proxy)
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
              if (lane == 0) mbar_arrive(&ctrl->wready[dg][st]);
            }
          }
        }
        __syncwarp();
        if (!early && ok && lane == 0) mbar_arrive(&ctrl->wempty[0]);
      }
    }
  } else {
    // ---- epilogue: warp quarter qd reads lanes 32 qd .. 32 qd + 31 (weight rows) of both accumulators ----
    const int qd = warp & 3;
    uint32_t tile_iter = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < a.n_tiles && ok; tile += gridDim.x, ++tile_iter) {
      const int tr = tile / a.MT, mt = tile % a.MT;
      const int halves = 2 * tr + 1 < a.MB ? 2 : 1;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(&ctrl->accfull, tile_iter & 1u, abortp, a.status));
      if (!ok) break;
      tc_fence_after();
      const int t0 = mt * kTileTokens;
      for (int h = 0; h < halves; ++h) {
        const int row = (2 * tr + h) * kTileRows + qd * 32 + lane;
#pragma unroll 1
        for (int cc = 0; cc < kTileTokens / 32; ++cc) {
          uint32_t r[32];
          tmem_ld32(tmem_base + (uint32_t)(h * kTileTokens + cc * 32) + ((uint32_t)(qd * 32) << 16), r);
          if (row < a.oc) {
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int t = t0 + cc * 32 + c;
              if (t < a.M) {
                if (a.y_dtype == RWKVQ_F32) static_cast<float*>(a.Y)[(size_t)t * a.oc + row] = __uint_as_float(r[c]);
                else static_cast<__nv_bfloat16*>(a.Y)[(size_t)t * a.oc + row] = __float2bfloat16_rn(__uint_as_float(r[c]));
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctrl->accempty);
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

extern "C" {

size_t rwkvq_prefill_workspace_bytes(const rwkvq_desc* d, int M, int has_mu) {
  (void)has_mu;   // the operand tiles are written whether or not a token shift is applied
  if (!d || M <= 0 || check_matrix_desc(d) != RWKVQ_OK) return 0;
  const size_t MT = ((size_t)M + pf::kTileTokens - 1) / pf::kTileTokens, KB = (size_t)d->ic_pad / pf::kKBlock;
  return MT * KB * pf::kXTileBytes;
}

rwkvq_status rwkvq_gemm_prefill(const rwkvq_desc* d, const void* W, const rwkvq_desc* mud, const void* mu, const void* X,
                                const void* xprev0, int M, void* Y, int y_dtype, void* ws, size_t ws_bytes, void* stream) {
  if (!d || !W || !X || !Y || M <= 0) return RWKVQ_EINVAL;
  if (y_dtype != RWKVQ_F32 && y_dtype != RWKVQ_BF16) return RWKVQ_EINVAL;
  if (mu && !mud) return RWKVQ_EINVAL;
  if (!mu && xprev0) return RWKVQ_EINVAL;
  if (d->oc == 1) return RWKVQ_ESHAPE;
  rwkvq_status st = check_matrix_desc(d);
  if (st != RWKVQ_OK) return st;
  if (mu) {
    st = check_vector_desc(mud, d->ic);
    if (st != RWKVQ_OK) return st;
  }
  if (d->ic % 8) return RWKVQ_ESHAPE;
  if (!aligned16(W) || !aligned16(X) || !aligned16(Y) || (mu && !aligned16(mu)) || (xprev0 && !aligned16(xprev0)) || (ws && !aligned16(ws)))
    return RWKVQ_EALIGN;
  const size_t need = rwkvq_prefill_workspace_bytes(d, M, mu != nullptr);
  if (!ws || ws_bytes < need) return RWKVQ_ENOMEM;
  if ((reinterpret_cast<uintptr_t>(ws) & 127u) != 0) return RWKVQ_EALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint8_t* img = static_cast<const uint8_t*>(W);
  pf::PrefillArgs a;
  a.payload = img + RWKVQ_HEADER_BYTES;
  a.aux = img + matrix_aux_offset(d);
  a.xtiles = static_cast<const uint8_t*>(ws);
  a.Y = Y;
  a.status = device_status_ptr();
  if (!a.status) return RWKVQ_ECUDA;
  a.oc = d->oc; a.ic = d->ic; a.M = M;
  a.KT = d->ic_pad / 256; a.KB = a.KT * 4; a.MB = d->oc_pad / 128;
  a.MT = (M + pf::kTileTokens - 1) / pf::kTileTokens;
  a.n_tiles = ((a.MB + 1) / 2) * a.MT;
  a.fmt = d->method == RWKVQ_SQ ? pf::PF_SQ3 : (d->bits == 6 ? pf::PF_VQ6 : pf::PF_VQ8);
  a.entries = d->entries; a.y_dtype = y_dtype;
  a.rec_bytes = d->method == RWKVQ_SQ ? (uint32_t)RWKVQ_SQ_RECORD_BYTES : rwkvq_vq_record_bytes(d->bits);
  a.chunk_bytes = 8u * a.rec_bytes;
  a.cb_bytes = d->method == RWKVQ_SQ ? 0u : (uint32_t)d->entries * 4u;
  // pre-pass
  const uint8_t* mup = nullptr; const uint8_t* mua = nullptr; int mu_bits = 0;
  if (mu) {
    const uint8_t* m = static_cast<const uint8_t*>(mu);
    mup = m + RWKVQ_HEADER_BYTES; mua = m + vector_aux_offset(mud); mu_bits = mud->bits;
  }
  const long long nvec = (long long)a.MT * pf::kTileTokens * a.KB * 8;
  pf::prefill_mix_kernel<<<(unsigned)((nvec + 255) / 256), 256, 0, s>>>(
      static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(xprev0), mup, mua, mu_bits, M, d->ic, a.KB, a.MT,
      static_cast<uint8_t*>(ws));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_status(e);
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  e = cudaFuncSetAttribute(pf::prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pf::kSmemBytes);
  if (e != cudaSuccess) return cuda_status(e);
  const int grid = a.n_tiles < sms ? a.n_tiles : sms;
  pf::prefill_kernel<<<grid, pf::kThreads, pf::kSmemBytes, s>>>(a);
  return cuda_status(cudaGetLastError());
}

}  // extern "C"
