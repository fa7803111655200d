// Device-side unpack routines shared by the decode product, the prefill product and the
// dequantisation probe.  Layout: see format.h.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "format.h"

namespace rwkvq {

// (a & MASK) | orv in one LOP3; the mask is an immediate of the instruction.
template <uint32_t MASK>
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t orv) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "n"(MASK), "r"(orv));
  return r;
}

// fp16 bit pattern of 2^(10-pos) replicated in both halves.
__host__ __device__ constexpr uint32_t sq_exp2(int pos) {
  return (uint32_t)((25 - pos) << 10) * 0x00010001u;
}

// One triple (three 32-bit words) -> sixteen half2 registers r[e], e = 4*m + R, each half
// holding q + (1024 >> rwkvq_sq_pos(e)) exactly.  21 integer instructions for 32 codes.
__device__ __forceinline__ void sq_unpack_triple(uint32_t wa, uint32_t wb, uint32_t wc, uint32_t (&r)[16]) {
  const uint32_t ua = wa >> 9, ub = wb >> 8, uc = wc >> 7;
  r[0] = and_or<0x00070007u>(wa, sq_exp2(0));
  r[1] = and_or<0x00380038u>(wa, sq_exp2(3));
  r[2] = and_or<0x01C001C0u>(wa, sq_exp2(6));
  r[3] = and_or<0x00070007u>(ua, sq_exp2(0));
  r[4] = and_or<0x00380038u>(ua, sq_exp2(3));
  r[5] = and_or<0x00070007u>(wb, sq_exp2(0));
  r[6] = and_or<0x00380038u>(wb, sq_exp2(3));
  r[7] = and_or<0x01C001C0u>(wb, sq_exp2(6));
  r[8] = and_or<0x000E000Eu>(ub, sq_exp2(1));
  r[9] = and_or<0x00700070u>(ub, sq_exp2(4));
  r[10] = and_or<0x00070007u>(wc, sq_exp2(0));
  r[11] = and_or<0x00380038u>(wc, sq_exp2(3));
  r[12] = and_or<0x01C001C0u>(wc, sq_exp2(6));
  r[13] = and_or<0x001C001Cu>(uc, sq_exp2(2));
  r[14] = and_or<0x00E000E0u>(uc, sq_exp2(5));
  uint32_t s = and_or<0x00400040u>(ua, sq_exp2(6));
  s = and_or<0x00800080u>(ub, s);
  r[15] = and_or<0x01000100u>(uc, s);
}

// Index n (0..63) of a lane's VQ stream of NW words; compile-time n folds the funnel shift.
template <int BITS, int NW>
__device__ __forceinline__ uint32_t vq_index(const uint32_t (&w)[NW], int n) {
  const int bit = BITS * n, wi = bit >> 5, sh = bit & 31;
  uint32_t v = (sh + BITS <= 32 || wi + 1 >= NW) ? (w[wi] >> sh) : __funnelshift_r(w[wi], w[wi + 1], sh);
  return v & ((1u << BITS) - 1u);
}

__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

}  // namespace rwkvq
