/*
 * Stateless counter-based generator for the synthetic benchmark inputs (host side, plain C).
 * Holds none of the method's arithmetic.  Element `index` of tensor `tensor_id` under `seed`
 * depends on nothing else, so any slice of a matrix can be regenerated on its own.
 *
 * kinds: 0 = N(0, p0) by Box-Muller, 1 = U(p0, p1), 2 = integers uniform in [-127, 127],
 *        3 = max(N(0, p0), 0).
 * dtype: 0 = fp16 bits, 1 = bf16 bits (both round-to-nearest-even), 2 = int8,
 *        3 = fp32 bits holding a TF32-representable value (10 mantissa bits, round-to-nearest-even),
 *        5 = fp8 e4m3 bits, 6 = fp8 e5m2 bits (round-to-nearest-even, saturating at the largest finite value).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

static uint64_t stream_key(uint64_t seed, uint64_t tensor_id, uint64_t stream) {
  return mix64(seed * 0x100000001B3ULL + tensor_id * 0x9E37ULL + stream * 0x51ED27ULL +
               0x9E3779B97F4A7C15ULL);
}

uint64_t sp24_inputs_raw(uint64_t seed, uint64_t tensor_id, uint64_t stream, uint64_t index) {
  return mix64(index * 0x9E3779B97F4A7C15ULL + stream_key(seed, tensor_id, stream));
}

static double unit_open(uint64_t u) { /* (0,1): 53 bits, offset by half a step */
  return ((double)(u >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

static uint16_t float_to_bf16_rne(float f) {
  uint32_t bits;
  memcpy(&bits, &f, 4);
  if ((bits & 0x7F800000u) == 0x7F800000u) return (uint16_t)(bits >> 16); /* inf / nan */
  bits += 0x7FFFu + ((bits >> 16) & 1u);
  return (uint16_t)(bits >> 16);
}

static uint32_t float_to_tf32_rne(float f) {
  uint32_t bits;
  memcpy(&bits, &f, 4);
  if ((bits & 0x7F800000u) == 0x7F800000u) return bits & 0xFFFFE000u;
  bits += 0xFFFu + ((bits >> 13) & 1u);
  return bits & 0xFFFFE000u;
}

static uint16_t double_to_half_rne(double d) {
  /* _Float16 conversion from double rounds once, to nearest even. */
  _Float16 h = (_Float16)d;
  uint16_t bits;
  memcpy(&bits, &h, 2);
  return bits;
}

/* 8-bit float with `mbits` mantissa bits and exponent bias `bias`; `max_bits` is the pattern of
 * the largest finite magnitude (results beyond it saturate there). */
static uint8_t double_to_fp8_rne(double d, int mbits, int bias, int max_bits) {
  uint8_t sign = signbit(d) ? 0x80 : 0;
  double a = fabs(d);
  int bits;
  if (a != a) return (uint8_t)(sign | 0x7F);
  if (a == 0.0) return sign;
  int e;
  frexp(a, &e); /* a = f * 2^e, f in [0.5, 1): unbiased exponent e - 1 */
  int E = e - 1;
  if (E < 1 - bias) {
    /* subnormal range: units of 2^(1 - bias - mbits); a carry into the first normal is the right pattern */
    bits = (int)rint(ldexp(a, -(1 - bias - mbits)));
  } else {
    int q = (int)rint(ldexp(a, mbits - E)); /* in [2^mbits, 2^(mbits+1)] */
    if (q == (2 << mbits)) { q >>= 1; ++E; }
    bits = ((E + bias) << mbits) | (q - (1 << mbits));
  }
  if (bits > max_bits) bits = max_bits;
  return (uint8_t)(sign | bits);
}

uint8_t sp24_inputs_to_fp8(double d, int e5m2) {
  return e5m2 ? double_to_fp8_rne(d, 2, 15, 0x7B) : double_to_fp8_rne(d, 3, 7, 0x7E);
}

void sp24_inputs_fill(int kind, double p0, double p1, int dtype, uint64_t seed,
                      uint64_t tensor_id, uint64_t start, uint64_t count, void* out) {
  const uint64_t k0 = stream_key(seed, tensor_id, 0), k1 = stream_key(seed, tensor_id, 1);
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < (int64_t)count; ++n) {
    uint64_t idx = (start + (uint64_t)n) * 0x9E3779B97F4A7C15ULL;
    uint64_t a = mix64(idx + k0);
    double v;
    if (kind == 2) {
      v = (double)((int)(a % 255u) - 127);
    } else if (kind == 1) {
      v = p0 + (p1 - p0) * unit_open(a);
    } else {
      uint64_t b = mix64(idx + k1);
      v = p0 * sqrt(-2.0 * log(unit_open(a))) * cos(6.283185307179586476925 * unit_open(b));
      if (kind == 3 && v < 0.0) v = 0.0;
    }
    if (dtype == 5 || dtype == 6) ((uint8_t*)out)[n] = sp24_inputs_to_fp8(v, dtype == 6);
    else if (dtype == 3) ((uint32_t*)out)[n] = float_to_tf32_rne((float)v);
    else if (dtype == 2) ((int8_t*)out)[n] = (int8_t)v;
    else if (dtype == 1) ((uint16_t*)out)[n] = float_to_bf16_rne((float)v);
    else ((uint16_t*)out)[n] = double_to_half_rne(v);
  }
}
