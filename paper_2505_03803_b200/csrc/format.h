// Physical layout of the packed device image, shared by the host packer and the kernels.
//
// Image = 256-byte header + payload.  The payload of a matrix is a grid of CHUNKS, one per
// (128-row block, 256-column tile), stored row-block-major: chunk(mb, kt) at
// payload + (mb * KT + kt) * chunk_bytes.  A chunk is 8 RECORDS, one per 16-row slice, and a
// record is what one warp consumes for sixteen m16n8k16 tensor-core steps: it is laid out
// lane-major in 512-byte planes (plane p, lane L -> 16 bytes), so that one 128-bit load per
// lane per plane is fully coalesced and the 32-bit words a lane receives are exactly the
// A-fragment registers' worth of codes of "its" two rows (g = L/4 and g+8) and columns.
//
// Column mapping inside a 256-column tile.  Tensor-core step j (0..15) covers columns
// 16j..16j+15.  Lane L = 4g + t holds, for step j, four fragment registers R = 0..3:
//     row  = g + 8 * (R & 1)
//     cols = 16j + 4t + 2 * (R >> 1) + {0, 1}        (low half = even column)
// so the matching B fragment of lane (g, t) is the 8 contiguous bytes x[n=g][16j+4t .. +3].
//
// SQ record (3-bit codes, group 128), 1664 bytes:
//   planes 0..2 (1536 B): 12 words per lane = 4 TRIPLES (A, B, C); triple i covers steps
//     4i..4i+3.  The 16 registers of a triple are numbered e = 4*m + R (m = step within the
//     triple).  Each 16-bit half of a word holds five 3-bit fields at bits 3f..3f+2 (f = 0..4)
//     and one spare bit 15; the low half is the even column, the high half the odd column.
//       e < 15 : word e / 5 of the triple, field e % 5
//       e = 15 : bit b of the code is the spare bit of word b (A, B, C)
//     Fields 0..2 are read in place, fields 3..4 after a right shift of 9 (A), 8 (B), 7 (C);
//     with those shifts the three spare bits land on adjacent mantissa bits 6, 7, 8, so that
//     every register is one LOP3 (mask | exponent) away from a half2 holding (q + bias) exactly.
//   plane 3 (128 B): for g = 0..7, 16 bytes = (s,z) fp16 pairs of (row g, group 0),
//     (row g, group 1), (row g+8, group 0), (row g+8, group 1); group = 128-column half of the tile.
//
// VQ record (2-D vectors, 6- or 8-bit indices), 1536 / 2048 bytes:
//   per lane 64 indices n = 4j + R, index n at bits [bits*n, bits*n + bits) of the lane's
//   little-endian bit stream of 12 / 16 words; planes as above.  The index of register R of
//   step j addresses the pair of columns given by the mapping above.  Codebooks live in the
//   aux area: [oc/256][ic/256][entries] half2.
//
// Vector image (token-shift mu, oc = 1): aux = one codebook; payload = ic/2 indices as a plain
//   little-endian bit stream in natural order.
#pragma once
#include <stdint.h>

#define RWKVQ_MAGIC 0x514B5752u /* "RWKQ" */
#define RWKVQ_VERSION 1u
#define RWKVQ_HEADER_BYTES 256

#define RWKVQ_ROWS_PER_RECORD 16
#define RWKVQ_RECORDS_PER_CHUNK 8
#define RWKVQ_CHUNK_ROWS 128
#define RWKVQ_TILE_COLS 256
#define RWKVQ_SQ_RECORD_BYTES 1664
#define RWKVQ_SQ_CODE_BYTES 1536

struct rwkvq_image_header {
  uint32_t magic, version;
  uint32_t method, bits;
  uint32_t oc, ic, oc_pad, ic_pad;
  uint32_t group, vec_dim, tile, entries;
  uint32_t record_bytes, chunk_bytes;
  uint32_t is_vector, reserved0;
  uint64_t off_payload, payload_bytes;
  uint64_t off_aux, aux_bytes;
  uint64_t image_bytes, stream_bytes;
  uint32_t crc32; /* of everything after the header */
  uint32_t reserved1;
  uint8_t pad[RWKVQ_HEADER_BYTES - 120];
};

#ifdef __cplusplus
static_assert(sizeof(rwkvq_image_header) == RWKVQ_HEADER_BYTES, "header size");
#endif

#define RWKVQ_IMAGE_FLAG_NO_CRC 1u /* reserved1 bit 0: the image was written on the device, crc32 is not set */

#if defined(__CUDACC__)
#define RWKVQ_HD __host__ __device__ inline
#else
#define RWKVQ_HD inline
#endif

// Mantissa bit position at which the 3-bit code of register e (0..15) of a triple appears
// after extraction; the half then holds q + (1024 >> pos) exactly.
RWKVQ_HD int rwkvq_sq_pos(int e) {
  if (e == 15) return 6;
  int wd = e / 5, f = e % 5;
  return f < 3 ? 3 * f : 3 * f - 9 + wd;
}
// Bias carried by column `o` (0..63) of a triple span, for row half h (0: rows g, 1: rows g+8).
RWKVQ_HD int rwkvq_sq_bias(int o, int h) {
  int m = o >> 4, R = (((o & 3) >> 1) << 1) | h;
  return 1024 >> rwkvq_sq_pos(4 * m + R);
}
RWKVQ_HD uint32_t rwkvq_vq_record_bytes(int bits) { return 64u * 32u * (uint32_t)bits / 8u; }

#ifdef __cplusplus
// Header of the image of a matrix (or vector) with these logical sizes; crc32 is left 0.
inline void rwkvq_fill_header(rwkvq_image_header* h, int method, int bits, int oc, int ic, int oc_pad, int ic_pad,
                              int group, int vec_dim, int tile, int entries, bool is_vector,
                              uint64_t image_bytes, uint64_t stream_bytes) {
  *h = rwkvq_image_header{};
  h->magic = RWKVQ_MAGIC; h->version = RWKVQ_VERSION;
  h->method = (uint32_t)method; h->bits = (uint32_t)bits; h->oc = (uint32_t)oc; h->ic = (uint32_t)ic;
  h->oc_pad = (uint32_t)oc_pad; h->ic_pad = (uint32_t)ic_pad;
  h->group = (uint32_t)group; h->vec_dim = (uint32_t)vec_dim; h->tile = (uint32_t)tile; h->entries = (uint32_t)entries;
  h->is_vector = is_vector ? 1u : 0u;
  h->off_payload = RWKVQ_HEADER_BYTES;
  h->image_bytes = image_bytes; h->stream_bytes = stream_bytes;
  if (method == 1) {            // SQ
    h->record_bytes = RWKVQ_SQ_RECORD_BYTES; h->chunk_bytes = 8 * RWKVQ_SQ_RECORD_BYTES;
    h->payload_bytes = (uint64_t)(oc_pad / 128) * (uint64_t)(ic_pad / 256) * h->chunk_bytes;
    h->aux_bytes = 0;
  } else if (!is_vector) {      // VQ matrix
    h->record_bytes = rwkvq_vq_record_bytes(bits); h->chunk_bytes = 8 * h->record_bytes;
    h->payload_bytes = (uint64_t)(oc / 128) * (uint64_t)(ic / 256) * h->chunk_bytes;
    h->aux_bytes = (uint64_t)(oc / 256) * (uint64_t)(ic / 256) * (uint64_t)entries * 4;
  } else {                      // VQ vector
    h->record_bytes = 0; h->chunk_bytes = 0;
    h->payload_bytes = ((((uint64_t)(ic / 2) * (uint64_t)bits + 7) / 8) + 15) / 16 * 16;
    h->aux_bytes = (uint64_t)entries * 4;
  }
  h->off_aux = h->off_payload + h->payload_bytes;
}
#endif
