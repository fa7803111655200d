// Host side of the library: quantizers (round-to-nearest group-wise SQ, Section 3.2 Eq. 2;
// k-means VQ, Section 3.2 Eq. 3), the bit packer that turns logical codes into the device
// image described in format.h, and its inverse.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/rwkvq.h"
#include "format.h"

struct rwkvq_blob {
  rwkvq_desc desc;
  bool is_vector;
  std::vector<uint8_t> q;          // logical codes / indices
  std::vector<uint16_t> scale, zero, codebook;
  std::vector<uint8_t> image;      // header + payload + aux
};

namespace {

// ---- fp16 <-> double, written out (IEEE binary16, round to nearest even) -------------------
double half_to_double(uint16_t h) {
  int sign = h >> 15, exp = (h >> 10) & 31, man = h & 1023;
  double v;
  if (exp == 0) v = std::ldexp((double)man, -24);
  else if (exp == 31) v = man ? NAN : INFINITY;
  else v = std::ldexp((double)(man + 1024), exp - 25);
  return sign ? -v : v;
}
uint16_t double_to_half(double d) {
  uint16_t sign = std::signbit(d) ? 0x8000 : 0;
  double a = std::fabs(d);
  if (std::isnan(d)) return 0x7E00;
  if (a >= 65520.0) return sign | 0x7C00;           // rounds to infinity
  if (a < std::ldexp(1.0, -25)) return sign;          // below half of the smallest subnormal
  int e;
  std::frexp(a, &e);                                  // a = f * 2^e, f in [0.5, 1)
  int exp = e - 1;                                    // a in [2^exp, 2^(exp+1))
  if (exp < -14) exp = -14;                           // subnormal range: fixed quantum 2^-24
  double q = std::ldexp(a, 10 - exp);                 // integer-valued after rounding
  double r = std::nearbyint(q);                       // default mode: nearest even
  uint32_t m = (uint32_t)r;
  if (exp == -14 && m < 1024) return sign | (uint16_t)m;               // subnormal (or rounds up to 1024)
  if (m == 2048) { m = 1024; exp += 1; }
  return sign | (uint16_t)(((exp + 15) << 10) + (m - 1024));
}

const float* half_table() {
  static float* table = [] {
    float* t = new float[65536];
    for (uint32_t i = 0; i < 65536; ++i) t[i] = (float)half_to_double((uint16_t)i);
    return t;
  }();
  return table;
}

uint32_t crc32_of(const uint8_t* p, size_t n) {
  static uint32_t table[256];
  static bool init = false;
  if (!init) {
    for (uint32_t i = 0; i < 256; ++i) {
      uint32_t c = i;
      for (int k = 0; k < 8; ++k) c = (c & 1) ? 0xEDB88320u ^ (c >> 1) : c >> 1;
      table[i] = c;
    }
    init = true;
  }
  uint32_t c = 0xFFFFFFFFu;
  for (size_t i = 0; i < n; ++i) c = table[(c ^ p[i]) & 255] ^ (c >> 8);
  return c ^ 0xFFFFFFFFu;
}

struct SplitMix64 {
  uint64_t s;
  explicit SplitMix64(uint64_t seed) : s(seed) {}
  uint64_t next() {
    uint64_t z = (s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  }
  double uniform() { return (double)(next() >> 11) * (1.0 / 9007199254740992.0); }
  size_t below(size_t n) { return (size_t)(uniform() * (double)n) % n; }
};

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- quantizers ------------------------------------------------------------------------------

// Eq. 2, one group.  `w` holds the group's weights as doubles (exact fp16 values).
void sq_encode_group(const double* w, int n, int qmax, uint8_t* q, uint16_t* s_out, uint16_t* z_out) {
  double mn = w[0], mx = w[0];
  for (int i = 1; i < n; ++i) { mn = std::min(mn, w[i]); mx = std::max(mx, w[i]); }
  uint16_t s16 = double_to_half((mx - mn) / (double)qmax);
  double s = half_to_double(s16);
  if (mx == mn || s == 0.0) {  // constant group c = min: exact codes
    double c = mn;
    *s_out = double_to_half(c == 0.0 ? 1.0 : std::fabs(c));
    *z_out = double_to_half(c < 0.0 ? 1.0 : 0.0);
    uint8_t code = c > 0.0 ? 1 : 0;
    for (int i = 0; i < n; ++i) q[i] = code;
    return;
  }
  double z = std::min((double)qmax, std::max(0.0, std::nearbyint(-mn / s)));
  for (int i = 0; i < n; ++i) {
    double v = std::nearbyint(w[i] / s) + z;
    q[i] = (uint8_t)std::min((double)qmax, std::max(0.0, v));
  }
  *s_out = s16;
  *z_out = double_to_half(z);
}

// k-means++ seeding and Lloyd iterations on n 2-D vectors; centres rounded to fp16 and the
// final assignment taken against the rounded centres (lowest index wins ties).
void kmeans2d(const float* vx, const float* vy, size_t n, int E, int iters, SplitMix64& rng,
              uint16_t* cb_out /*[E][2]*/, uint8_t* idx_out) {
  std::vector<double> cx(E), cy(E), dist(n);
  size_t first = rng.below(n);
  cx[0] = vx[first]; cy[0] = vy[first];
  for (size_t i = 0; i < n; ++i) {
    double dx = vx[i] - cx[0], dy = vy[i] - cy[0];
    dist[i] = dx * dx + dy * dy;
  }
  for (int e = 1; e < E; ++e) {
    double tot = 0.0;
    for (size_t i = 0; i < n; ++i) tot += dist[i];
    size_t pick = 0;
    if (tot > 0.0) {
      double target = rng.uniform() * tot, acc = 0.0;
      pick = n - 1;
      for (size_t i = 0; i < n; ++i) { acc += dist[i]; if (acc > target) { pick = i; break; } }
    } else {
      pick = rng.below(n);
    }
    cx[e] = vx[pick]; cy[e] = vy[pick];
    for (size_t i = 0; i < n; ++i) {
      double dx = vx[i] - cx[e], dy = vy[i] - cy[e];
      dist[i] = std::min(dist[i], dx * dx + dy * dy);
    }
  }
  std::vector<float> fx(E), fy(E);
  std::vector<double> sx(E), sy(E);
  std::vector<size_t> cnt(E);
  auto assign = [&](size_t i) {
    float best = INFINITY; int bi = 0;
    float x = vx[i], y = vy[i];
    for (int e = 0; e < E; ++e) {
      float dx = x - fx[e], dy = y - fy[e];
      float d = dx * dx + dy * dy;
      if (d < best) { best = d; bi = e; }
    }
    return bi;
  };
  for (int it = 0; it < iters; ++it) {
    for (int e = 0; e < E; ++e) { fx[e] = (float)cx[e]; fy[e] = (float)cy[e]; sx[e] = sy[e] = 0.0; cnt[e] = 0; }
    for (size_t i = 0; i < n; ++i) {
      int bi = assign(i);
      sx[bi] += vx[i]; sy[bi] += vy[i]; cnt[bi]++;
    }
    for (int e = 0; e < E; ++e)
      if (cnt[e]) { cx[e] = sx[e] / (double)cnt[e]; cy[e] = sy[e] / (double)cnt[e]; }
  }
  std::vector<double> hx(E), hy(E);
  for (int e = 0; e < E; ++e) {
    cb_out[2 * e] = double_to_half(cx[e]);
    cb_out[2 * e + 1] = double_to_half(cy[e]);
    hx[e] = half_to_double(cb_out[2 * e]);
    hy[e] = half_to_double(cb_out[2 * e + 1]);
  }
  for (size_t i = 0; i < n; ++i) {  // final assignment in double: exact on fp16 data
    double best = INFINITY; int bi = 0;
    for (int e = 0; e < E; ++e) {
      double dx = (double)vx[i] - hx[e], dy = (double)vy[i] - hy[e];
      double d = dx * dx + dy * dy;
      if (d < best) { best = d; bi = e; }
    }
    idx_out[i] = (uint8_t)bi;
  }
}

// ---- bit packing -----------------------------------------------------------------------------

inline void put_bits(uint8_t* base, size_t bitpos, uint32_t value, int nbits) {
  for (int b = 0; b < nbits; ++b)
    if ((value >> b) & 1u) base[(bitpos + b) >> 3] |= (uint8_t)(1u << ((bitpos + b) & 7));
}
inline uint32_t get_bits(const uint8_t* base, size_t bitpos, int nbits) {
  uint32_t v = 0;
  for (int b = 0; b < nbits; ++b) v |= (uint32_t)((base[(bitpos + b) >> 3] >> ((bitpos + b) & 7)) & 1u) << b;
  return v;
}
// Byte offset, inside a record, of word `widx` of lane L (planes of 512 bytes).
inline size_t lane_word_off(int L, int widx) { return (size_t)(widx >> 2) * 512 + (size_t)L * 16 + (size_t)(widx & 3) * 4; }

// Fast path of the packer: builds the three words of each triple directly.
void sq_record_pack_fast(uint8_t* rec, const uint8_t* q, int ic, int oc, int r0, int c0) {
  for (int L = 0; L < 32; ++L) {
    const int g = L >> 2, t = L & 3;
    for (int i = 0; i < 4; ++i) {
      uint32_t w3[3] = {0u, 0u, 0u};
      for (int e = 0; e < 16; ++e) {
        const int m = e >> 2, R = e & 3;
        const int row = r0 + g + 8 * (R & 1);
        const int col = c0 + 64 * i + 16 * m + 4 * t + 2 * (R >> 1);
        uint32_t lo = 0, hi = 0;
        if (row < oc && col < ic) { lo = q[(size_t)row * ic + col]; hi = q[(size_t)row * ic + col + 1]; }
        const uint32_t pair = lo | (hi << 16);
        if (e < 15) {
          w3[e / 5] |= pair << (3 * (e % 5));
        } else {
          for (int b = 0; b < 3; ++b) w3[b] |= ((pair >> b) & 0x00010001u) << 15;
        }
      }
      for (int wd = 0; wd < 3; ++wd) std::memcpy(rec + lane_word_off(L, 3 * i + wd), &w3[wd], 4);
    }
  }
}

void vq_record_pack_fast(uint8_t* rec, const uint8_t* idx, int bits, int half_ic, int r0, int p0) {
  const int nw = 2 * bits;
  for (int L = 0; L < 32; ++L) {
    const int g = L >> 2, t = L & 3;
    uint32_t words[17] = {0};
    for (int n = 0; n < 64; ++n) {
      const int j = n >> 2, R = n & 3;
      const int row = r0 + g + 8 * (R & 1);
      const int pair = p0 + 8 * j + 2 * t + (R >> 1);
      const uint32_t v = idx[(size_t)row * half_ic + pair];
      const int bitpos = bits * n, wi = bitpos >> 5, sh = bitpos & 31;
      words[wi] |= v << sh;
      if (sh + bits > 32) words[wi + 1] |= v >> (32 - sh);
    }
    for (int wi = 0; wi < nw; ++wi) std::memcpy(rec + lane_word_off(L, wi), &words[wi], 4);
  }
}

// Visit every (row, column) of an SQ record with the place its code lives.
// pack == true writes codes from q into rec; pack == false reads them back.
void sq_record_codes(uint8_t* rec, uint8_t* q, int ic, int oc, int r0, int c0, bool pack) {
  for (int L = 0; L < 32; ++L) {
    int g = L >> 2, t = L & 3;
    for (int i = 0; i < 4; ++i) {
      for (int e = 0; e < 16; ++e) {
        int m = e >> 2, R = e & 3;
        int row = r0 + g + 8 * (R & 1);
        int col = c0 + 64 * i + 16 * m + 4 * t + 2 * (R >> 1);
        for (int hf = 0; hf < 2; ++hf) {
          bool inside = row < oc && col + hf < ic;
          uint32_t code = (pack && inside) ? q[(size_t)row * ic + col + hf] : 0;
          if (e < 15) {
            int wd = e / 5, f = e % 5;
            size_t bit = lane_word_off(L, 3 * i + wd) * 8 + 16 * hf + 3 * f;
            if (pack) put_bits(rec, bit, code, 3); else code = get_bits(rec, bit, 3);
          } else {
            code = pack ? code : 0;
            for (int b = 0; b < 3; ++b) {
              size_t bit = lane_word_off(L, 3 * i + b) * 8 + 16 * hf + 15;
              if (pack) put_bits(rec, bit, (code >> b) & 1u, 1); else code |= get_bits(rec, bit, 1) << b;
            }
          }
          if (!pack && inside) q[(size_t)row * ic + col + hf] = (uint8_t)code;
        }
      }
    }
  }
}

void vq_record_codes(uint8_t* rec, uint8_t* idx, int bits, int half_ic, int r0, int p0, bool pack) {
  for (int L = 0; L < 32; ++L) {
    int g = L >> 2, t = L & 3;
    for (int n = 0; n < 64; ++n) {
      int j = n >> 2, R = n & 3;
      int row = r0 + g + 8 * (R & 1);
      int pair = p0 + 8 * j + 2 * t + (R >> 1);
      size_t bitpos = (size_t)bits * n;
      int widx = (int)(bitpos >> 5);
      int inword = (int)(bitpos & 31);
      // the field may straddle two words of the lane's stream
      uint32_t v = pack ? idx[(size_t)row * half_ic + pair] : 0;
      for (int b = 0; b < bits; ++b) {
        int wi = widx + ((inword + b) >> 5), bi = (inword + b) & 31;
        size_t bit = lane_word_off(L, wi) * 8 + bi;
        if (pack) put_bits(rec, bit, (v >> b) & 1u, 1); else v |= get_bits(rec, bit, 1) << b;
      }
      if (!pack) idx[(size_t)row * half_ic + pair] = (uint8_t)v;
    }
  }
}

rwkvq_status fill_desc(rwkvq_desc* d, int method, int bits, int oc, int ic, int group, int tile, bool is_vector) {
  std::memset(d, 0, sizeof(*d));
  d->method = method; d->bits = bits; d->oc = oc; d->ic = ic;
  if (method == RWKVQ_SQ) {
    if (bits != 3) return RWKVQ_EUNSUPPORTED;
    if (group != 128) return RWKVQ_EUNSUPPORTED;
    if (oc <= 0 || ic <= 0 || oc % 16 || ic % 128) return RWKVQ_ESHAPE;
    d->group = 128; d->vec_dim = 1; d->tile = 0; d->entries = 0;
    d->oc_pad = (int)round_up(oc, RWKVQ_CHUNK_ROWS); d->ic_pad = (int)round_up(ic, RWKVQ_TILE_COLS);
    size_t chunks = (size_t)(d->oc_pad / 128) * (d->ic_pad / 256);
    d->stream_bytes = chunks * 8 * RWKVQ_SQ_RECORD_BYTES;
    d->image_bytes = RWKVQ_HEADER_BYTES + d->stream_bytes;
  } else if (method == RWKVQ_VQ) {
    if (bits != 6 && bits != 8) return RWKVQ_EUNSUPPORTED;
    d->group = 0; d->vec_dim = 2; d->entries = 1 << bits;
    if (is_vector) {
      if (oc != 1 || ic <= 0 || ic % 2) return RWKVQ_ESHAPE;
      d->tile = 0; d->oc_pad = 1; d->ic_pad = ic;
      size_t idx_bytes = round_up(((size_t)(ic / 2) * bits + 7) / 8, 16);
      d->stream_bytes = idx_bytes + (size_t)d->entries * 4;
      d->image_bytes = round_up(RWKVQ_HEADER_BYTES + d->stream_bytes, 256);
    } else {
      if (tile != 256) return RWKVQ_EUNSUPPORTED;
      if (oc <= 0 || ic <= 0 || oc % 256 || ic % 256) return RWKVQ_ESHAPE;
      d->tile = 256; d->oc_pad = oc; d->ic_pad = ic;
      size_t chunks = (size_t)(oc / 128) * (ic / 256);
      size_t cb = (size_t)(oc / 256) * (ic / 256) * d->entries * 4;
      d->stream_bytes = chunks * 8 * rwkvq_vq_record_bytes(bits) + cb;
      d->image_bytes = round_up(RWKVQ_HEADER_BYTES + d->stream_bytes, 256);
    }
  } else {
    return RWKVQ_EINVAL;
  }
  return RWKVQ_OK;
}

void build_image(rwkvq_blob* b) {
  const rwkvq_desc& d = b->desc;
  b->image.assign(d.image_bytes, 0);
  rwkvq_image_header h;
  rwkvq_fill_header(&h, d.method, d.bits, d.oc, d.ic, d.oc_pad, d.ic_pad, d.group, d.vec_dim, d.tile, d.entries,
                    b->is_vector, d.image_bytes, d.stream_bytes);
  uint8_t* img = b->image.data();
  if (d.method == RWKVQ_SQ) {
    int MB = d.oc_pad / 128, KT = d.ic_pad / 256, ng = d.ic / 128;
#pragma omp parallel for collapse(2) schedule(static)
    for (int mb = 0; mb < MB; ++mb)
      for (int kt = 0; kt < KT; ++kt)
        for (int rt = 0; rt < 8; ++rt) {
          uint8_t* rec = img + h.off_payload + ((size_t)(mb * KT + kt) * 8 + rt) * RWKVQ_SQ_RECORD_BYTES;
          int r0 = mb * 128 + rt * 16, c0 = kt * 256;
          sq_record_pack_fast(rec, b->q.data(), d.ic, d.oc, r0, c0);
          uint16_t* sz = reinterpret_cast<uint16_t*>(rec + RWKVQ_SQ_CODE_BYTES);
          for (int g = 0; g < 8; ++g)
            for (int k = 0; k < 4; ++k) {
              int row = r0 + g + 8 * (k >> 1), grp = kt * 2 + (k & 1);
              bool inside = row < d.oc && grp < ng;
              sz[g * 8 + k * 2] = inside ? b->scale[(size_t)row * ng + grp] : 0;
              sz[g * 8 + k * 2 + 1] = inside ? b->zero[(size_t)row * ng + grp] : 0;
            }
        }
  } else if (!b->is_vector) {
    uint32_t rb = rwkvq_vq_record_bytes(d.bits);
    int MB = d.oc / 128, KT = d.ic / 256;
#pragma omp parallel for collapse(2) schedule(static)
    for (int mb = 0; mb < MB; ++mb)
      for (int kt = 0; kt < KT; ++kt)
        for (int rt = 0; rt < 8; ++rt) {
          uint8_t* rec = img + h.off_payload + ((size_t)(mb * KT + kt) * 8 + rt) * rb;
          vq_record_pack_fast(rec, b->q.data(), d.bits, d.ic / 2, mb * 128 + rt * 16, kt * 128);
        }
    std::memcpy(img + h.off_aux, b->codebook.data(), h.aux_bytes);
  } else {
    for (int p = 0; p < d.ic / 2; ++p) put_bits(img + h.off_payload, (size_t)p * d.bits, b->q[p], d.bits);
    std::memcpy(img + h.off_aux, b->codebook.data(), h.aux_bytes);
  }
  h.crc32 = crc32_of(img + RWKVQ_HEADER_BYTES, d.image_bytes - RWKVQ_HEADER_BYTES);
  std::memcpy(img, &h, sizeof(h));
}

size_t n_groups(const rwkvq_desc& d) { return (size_t)d.oc * (d.ic / 128); }
size_t n_codebook_halves(const rwkvq_desc& d, bool is_vector) {
  return is_vector ? (size_t)d.entries * 2 : (size_t)(d.oc / 256) * (d.ic / 256) * d.entries * 2;
}

}  // namespace

extern "C" {

rwkvq_status rwkvq_pack(const uint16_t* w, int oc, int ic, const rwkvq_quant_cfg* cfg, rwkvq_blob** out) {
  if (!cfg || !out) return RWKVQ_EINVAL;
  *out = nullptr;
  if (!w && !cfg->codes_in) return RWKVQ_EINVAL;
  bool is_vector = (cfg->method == RWKVQ_VQ && oc == 1);
  rwkvq_blob* b = new (std::nothrow) rwkvq_blob();
  if (!b) return RWKVQ_ENOMEM;
  b->is_vector = is_vector;
  rwkvq_status st = fill_desc(&b->desc, cfg->method, cfg->bits, oc, ic, cfg->group, cfg->tile, is_vector);
  if (st == RWKVQ_OK && cfg->method == RWKVQ_VQ && cfg->vec_dim != 2) st = RWKVQ_EUNSUPPORTED;
  if (st != RWKVQ_OK) { delete b; return st; }
  const rwkvq_desc& d = b->desc;
  try {
    if (w && !cfg->codes_in) {
      const size_t n = (size_t)oc * ic;
      volatile bool bad = false;
#pragma omp parallel for schedule(static)
      for (long long i = 0; i < (long long)n; ++i)
        if ((w[i] & 0x7C00) == 0x7C00) bad = true;
      if (bad) { delete b; return RWKVQ_ENONFINITE; }
    }
    if (cfg->method == RWKVQ_SQ) {
      size_t ng = n_groups(d);
      b->q.resize((size_t)oc * ic); b->scale.resize(ng); b->zero.resize(ng);
      if (cfg->codes_in) {
        const rwkvq_codes* c = cfg->codes_in;
        if (!c->q || !c->scale || !c->zero) { delete b; return RWKVQ_EINVAL; }
        for (size_t i = 0; i < b->q.size(); ++i) if (c->q[i] > 7) { delete b; return RWKVQ_EINVAL; }
        std::memcpy(b->q.data(), c->q, b->q.size());
        std::memcpy(b->scale.data(), c->scale, ng * 2);
        std::memcpy(b->zero.data(), c->zero, ng * 2);
      } else {
        const int gpr = ic / 128;
        const float* ht = half_table();
#pragma omp parallel for schedule(static)
        for (long long gi = 0; gi < (long long)ng; ++gi) {
          size_t row = gi / gpr, grp = gi % gpr;
          double tmp[128];
          const uint16_t* src = w + row * ic + grp * 128;
          for (int i = 0; i < 128; ++i) tmp[i] = (double)ht[src[i]];
          sq_encode_group(tmp, 128, 7, b->q.data() + row * ic + grp * 128, &b->scale[gi], &b->zero[gi]);
        }
      }
    } else {
      size_t nidx = (size_t)oc * ic / 2, ncb = n_codebook_halves(d, is_vector);
      b->q.resize(nidx); b->codebook.resize(ncb);
      if (cfg->codes_in) {
        const rwkvq_codes* c = cfg->codes_in;
        if (!c->q || !c->codebook) { delete b; return RWKVQ_EINVAL; }
        for (size_t i = 0; i < nidx; ++i) if ((int)c->q[i] >= d.entries) { delete b; return RWKVQ_EINVAL; }
        std::memcpy(b->q.data(), c->q, nidx);
        std::memcpy(b->codebook.data(), c->codebook, ncb * 2);
      } else if (is_vector) {
        std::vector<float> vx(ic / 2), vy(ic / 2);
        for (int p = 0; p < ic / 2; ++p) { vx[p] = (float)half_to_double(w[2 * p]); vy[p] = (float)half_to_double(w[2 * p + 1]); }
        SplitMix64 rng(cfg->seed);
        kmeans2d(vx.data(), vy.data(), ic / 2, d.entries, cfg->kmeans_iters, rng, b->codebook.data(), b->q.data());
      } else {
        const int TR = oc / 256, TC = ic / 256;
        const float* ht = half_table();
#pragma omp parallel for collapse(2) schedule(dynamic)
        for (int tr = 0; tr < TR; ++tr)
          for (int tc = 0; tc < TC; ++tc) {
            std::vector<float> vx(256 * 128), vy(256 * 128);
            std::vector<uint8_t> ix(256 * 128);
            for (int r = 0; r < 256; ++r)
              for (int p = 0; p < 128; ++p) {
                const uint16_t* src = w + (size_t)(tr * 256 + r) * ic + tc * 256 + 2 * p;
                vx[r * 128 + p] = ht[src[0]];
                vy[r * 128 + p] = ht[src[1]];
              }
            SplitMix64 rng(cfg->seed * 0x9E3779B97F4A7C15ull + (uint64_t)(tr * TC + tc) + 1);
            kmeans2d(vx.data(), vy.data(), 256 * 128, d.entries, cfg->kmeans_iters, rng,
                     b->codebook.data() + (size_t)(tr * TC + tc) * d.entries * 2, ix.data());
            for (int r = 0; r < 256; ++r)
              std::memcpy(b->q.data() + (size_t)(tr * 256 + r) * (ic / 2) + tc * 128, ix.data() + r * 128, 128);
          }
      }
    }
    build_image(b);
  } catch (const std::bad_alloc&) {
    delete b;
    return RWKVQ_ENOMEM;
  }
  *out = b;
  return RWKVQ_OK;
}

rwkvq_status rwkvq_desc_for(const rwkvq_quant_cfg* cfg, int oc, int ic, rwkvq_desc* desc_out) {
  if (!cfg || !desc_out) return RWKVQ_EINVAL;
  rwkvq_status st = fill_desc(desc_out, cfg->method, cfg->bits, oc, ic, cfg->group, cfg->tile,
                              cfg->method == RWKVQ_VQ && oc == 1);
  if (st == RWKVQ_OK && cfg->method == RWKVQ_VQ && cfg->vec_dim != 2) st = RWKVQ_EUNSUPPORTED;
  return st;
}

rwkvq_status rwkvq_blob_desc(const rwkvq_blob* b, rwkvq_desc* d) {
  if (!b || !d) return RWKVQ_EINVAL;
  *d = b->desc;
  return RWKVQ_OK;
}
size_t rwkvq_blob_nbytes(const rwkvq_blob* b) { return b ? b->image.size() : 0; }
rwkvq_status rwkvq_blob_image(const rwkvq_blob* b, void* dst, size_t n) {
  if (!b || !dst) return RWKVQ_EINVAL;
  if (n < b->image.size()) return RWKVQ_ENOMEM;
  std::memcpy(dst, b->image.data(), b->image.size());
  return RWKVQ_OK;
}
rwkvq_status rwkvq_blob_export_codes(const rwkvq_blob* b, rwkvq_codes* dst) {
  if (!b || !dst || !dst->q) return RWKVQ_EINVAL;
  std::memcpy(dst->q, b->q.data(), b->q.size());
  if (b->desc.method == RWKVQ_SQ) {
    if (!dst->scale || !dst->zero) return RWKVQ_EINVAL;
    std::memcpy(dst->scale, b->scale.data(), b->scale.size() * 2);
    std::memcpy(dst->zero, b->zero.data(), b->zero.size() * 2);
  } else {
    if (!dst->codebook) return RWKVQ_EINVAL;
    std::memcpy(dst->codebook, b->codebook.data(), b->codebook.size() * 2);
  }
  return RWKVQ_OK;
}

rwkvq_status rwkvq_image_unpack(const void* image, size_t n, rwkvq_desc* desc_out, rwkvq_codes* dst) {
  if (!image || n < RWKVQ_HEADER_BYTES) return RWKVQ_EINVAL;
  rwkvq_image_header h;
  std::memcpy(&h, image, sizeof(h));
  if (h.magic != RWKVQ_MAGIC || h.version != RWKVQ_VERSION) return RWKVQ_EINVAL;
  rwkvq_desc d;
  rwkvq_status st = fill_desc(&d, (int)h.method, (int)h.bits, (int)h.oc, (int)h.ic, (int)h.group, (int)h.tile, h.is_vector != 0);
  if (st != RWKVQ_OK) return st;
  if (d.image_bytes != h.image_bytes || n < d.image_bytes) return RWKVQ_EINVAL;
  const uint8_t* img = static_cast<const uint8_t*>(image);
  if (!(h.reserved1 & RWKVQ_IMAGE_FLAG_NO_CRC) &&
      crc32_of(img + RWKVQ_HEADER_BYTES, d.image_bytes - RWKVQ_HEADER_BYTES) != h.crc32) return RWKVQ_EINVAL;
  {  // offsets come from the logical sizes, never from the header bytes
    rwkvq_image_header ref;
    rwkvq_fill_header(&ref, d.method, d.bits, d.oc, d.ic, d.oc_pad, d.ic_pad, d.group, d.vec_dim, d.tile, d.entries,
                      h.is_vector != 0, d.image_bytes, d.stream_bytes);
    if (ref.off_payload != h.off_payload || ref.off_aux != h.off_aux || ref.aux_bytes != h.aux_bytes ||
        ref.off_aux + ref.aux_bytes > d.image_bytes) return RWKVQ_EINVAL;
  }
  if (desc_out) *desc_out = d;
  if (!dst) return RWKVQ_OK;
  if (!dst->q) return RWKVQ_EINVAL;
  uint8_t* mut = const_cast<uint8_t*>(img);  // the visitors only read when pack == false
  if (d.method == RWKVQ_SQ) {
    if (!dst->scale || !dst->zero) return RWKVQ_EINVAL;
    int MB = d.oc_pad / 128, KT = d.ic_pad / 256, ng = d.ic / 128;
    for (int mb = 0; mb < MB; ++mb)
      for (int kt = 0; kt < KT; ++kt)
        for (int rt = 0; rt < 8; ++rt) {
          uint8_t* rec = mut + h.off_payload + ((size_t)(mb * KT + kt) * 8 + rt) * RWKVQ_SQ_RECORD_BYTES;
          int r0 = mb * 128 + rt * 16;
          sq_record_codes(rec, dst->q, d.ic, d.oc, r0, kt * 256, false);
          const uint16_t* sz = reinterpret_cast<const uint16_t*>(rec + RWKVQ_SQ_CODE_BYTES);
          for (int g = 0; g < 8; ++g)
            for (int k = 0; k < 4; ++k) {
              int row = r0 + g + 8 * (k >> 1), grp = kt * 2 + (k & 1);
              if (row < d.oc && grp < ng) {
                dst->scale[(size_t)row * ng + grp] = sz[g * 8 + k * 2];
                dst->zero[(size_t)row * ng + grp] = sz[g * 8 + k * 2 + 1];
              }
            }
        }
  } else {
    if (!dst->codebook) return RWKVQ_EINVAL;
    if (h.is_vector) {
      for (int p = 0; p < d.ic / 2; ++p) dst->q[p] = (uint8_t)get_bits(img + h.off_payload, (size_t)p * d.bits, d.bits);
    } else {
      int MB = d.oc / 128, KT = d.ic / 256;
      uint32_t rb = rwkvq_vq_record_bytes(d.bits);
      for (int mb = 0; mb < MB; ++mb)
        for (int kt = 0; kt < KT; ++kt)
          for (int rt = 0; rt < 8; ++rt) {
            uint8_t* rec = mut + h.off_payload + ((size_t)(mb * KT + kt) * 8 + rt) * rb;
            vq_record_codes(rec, dst->q, d.bits, d.ic / 2, mb * 128 + rt * 16, kt * 128, false);
          }
    }
    std::memcpy(dst->codebook, img + h.off_aux, h.aux_bytes);
  }
  return RWKVQ_OK;
}

void rwkvq_blob_free(rwkvq_blob* b) { delete b; }

const char* rwkvq_status_str(rwkvq_status s) {
  switch (s) {
    case RWKVQ_OK: return "ok";
    case RWKVQ_EINVAL: return "invalid argument";
    case RWKVQ_ESHAPE: return "unsupported shape";
    case RWKVQ_EALIGN: return "misaligned pointer";
    case RWKVQ_ENONFINITE: return "non-finite weight";
    case RWKVQ_ENOMEM: return "out of memory or buffer too small";
    case RWKVQ_ECUDA: return "CUDA error";
    case RWKVQ_EUNSUPPORTED: return "unsupported configuration";
    case RWKVQ_ETIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

}  // extern "C"
