/*
 * CPU oracle for the 2:4 structured-sparse path of "Accelerating Sparse Deep Neural
 * Networks" (arXiv 2104.08378).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, scalar restatement of
 * what the path computes, written from the paper, and shares no code with the CUDA library.
 * Only the tests, the smoke check and the bench's CPU-baseline / reference legs may call it.
 *
 * Every function walks the definition directly: one loop per index, no blocking, no fusion.
 * Floating-point GEMMs read the fp16 / bf16 inputs exactly into double and accumulate in
 * double; the int8 GEMM accumulates in int64.  The only concession to run time is an OpenMP
 * "parallel for" over output rows (rows are independent in every operation here).
 *
 * dtype codes: 0 = fp16, 1 = bf16, 2 = int8, 5 = fp8 e4m3, 6 = fp8 e5m2 (the 8-bit floating-point
 * types are not in the paper: same 2:4 pattern and format, OCP 8-bit floating-point encodings).
 * Matrices are row-major with a leading dimension in elements unless stated.
 *
 * Pins (tests/test_oracle_*.py): the pattern invariant and idempotence, brute force over all
 * C(4,2) keep-patterns, the metadata example of Section 3.1, the storage arithmetic of
 * Section 3.1, decompress(compress(x)) == prune(x), sparse GEMM == library dense matmul on
 * the pruned matrix, closed forms (identity B, all-ones), a direct 7-loop convolution for
 * im2col, hand-computed positions for the tensor-core metadata permutation, and for the
 * error-bound scale (|A| . |B|) a library matmul of the magnitudes plus its closed forms.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------------------- */
/* element helpers                                                                       */
/* ------------------------------------------------------------------------------------- */

static int elem_size(int dtype) { return (dtype == 2 || dtype == 5 || dtype == 6) ? 1 : 2; }
static int is_fp8(int dtype) { return dtype == 5 || dtype == 6; }

/* IEEE binary16 bit pattern -> double, exactly. */
static double half_bits_to_double(uint16_t h) {
  int sign = (h >> 15) & 1;
  int exponent = (h >> 10) & 0x1F;
  int mantissa = h & 0x3FF;
  double v;
  if (exponent == 0) {
    v = ldexp((double)mantissa, -24); /* zero and subnormals: mantissa * 2^-24 */
  } else if (exponent == 31) {
    v = mantissa ? NAN : INFINITY;
  } else {
    v = ldexp((double)(mantissa + 1024), exponent - 25); /* (1 + m/1024) * 2^(e-15) */
  }
  return sign ? -v : v;
}

/* bfloat16 bit pattern -> double, exactly: bf16 is the upper half of an IEEE binary32. */
static double bf16_bits_to_double(uint16_t b) {
  uint32_t w = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &w, sizeof f);
  return (double)f;
}

/* 8-bit floating point, e4m3: 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinities, the
 * single NaN pattern per sign is exponent and mantissa all ones; largest finite value 448. */
static double e4m3_bits_to_double(uint8_t b) {
  int sign = (b >> 7) & 1;
  int exponent = (b >> 3) & 0xF;
  int mantissa = b & 0x7;
  double v;
  if (exponent == 15 && mantissa == 7) v = NAN;
  else if (exponent == 0) v = ldexp((double)mantissa, -9); /* m/8 * 2^-6 */
  else v = ldexp((double)(mantissa + 8), exponent - 10);   /* (1 + m/8) * 2^(e-7) */
  return sign ? -v : v;
}

/* 8-bit floating point, e5m2: 1 sign, 5 exponent (bias 15), 2 mantissa bits; IEEE-style
 * infinities and NaNs. */
static double e5m2_bits_to_double(uint8_t b) {
  int sign = (b >> 7) & 1;
  int exponent = (b >> 2) & 0x1F;
  int mantissa = b & 0x3;
  double v;
  if (exponent == 31) v = mantissa ? NAN : INFINITY;
  else if (exponent == 0) v = ldexp((double)mantissa, -16); /* m/4 * 2^-14 */
  else v = ldexp((double)(mantissa + 4), exponent - 17);    /* (1 + m/4) * 2^(e-15) */
  return sign ? -v : v;
}

static double load_as_double(int dtype, const void* base, int64_t index) {
  if (dtype == 5) return e4m3_bits_to_double(((const uint8_t*)base)[index]);
  if (dtype == 6) return e5m2_bits_to_double(((const uint8_t*)base)[index]);
  if (dtype == 0) return half_bits_to_double(((const uint16_t*)base)[index]);
  if (dtype == 1) return bf16_bits_to_double(((const uint16_t*)base)[index]);
  return (double)((const int8_t*)base)[index];
}

/* Magnitude key used by the pruning criterion (Section 4.1, step 2).
 * 16-bit floats: the bit pattern without the sign bit, which orders finite values by |x|
 * (zero of either sign -> 0, subnormals keep their rank).  int8: |x| as an int, -128 -> 128.
 * 8-bit floats: the seven bits below the sign, same argument as for the 16-bit floats. */
static int magnitude_key(int dtype, const void* base, int64_t index) {
  if (is_fp8(dtype)) return ((const uint8_t*)base)[index] & 0x7F;
  if (dtype == 2) {
    int v = ((const int8_t*)base)[index];
    return v < 0 ? -v : v;
  }
  return ((const uint16_t*)base)[index] & 0x7FFF;
}

/* The two kept positions of one group of four (Section 4.1 step 2: the two smallest are
 * removed; ties keep the lower index).  Rank each position by how many others beat it: j
 * beats p if its key is larger, or equal with a smaller index.  Positions with rank 0 and 1
 * are kept; they are returned in ascending order p0 < p1 (Section 3.1 lists indices in
 * ascending order inside a group). */
static void select_two(const int key[4], int* p0, int* p1) {
  int kept[2];
  int n = 0;
  for (int p = 0; p < 4; ++p) {
    int beaten_by = 0;
    for (int j = 0; j < 4; ++j) {
      if (j == p) continue;
      if (key[j] > key[p] || (key[j] == key[p] && j < p)) ++beaten_by;
    }
    if (beaten_by < 2) kept[n++] = p;
  }
  *p0 = kept[0];
  *p1 = kept[1];
}

static void copy_elem(int dtype, void* dst, int64_t di, const void* src, int64_t si) {
  if (elem_size(dtype) == 1) ((int8_t*)dst)[di] = ((const int8_t*)src)[si];
  else ((uint16_t*)dst)[di] = ((const uint16_t*)src)[si];
}

static void zero_elem(int dtype, void* dst, int64_t di) {
  if (elem_size(dtype) == 1) ((int8_t*)dst)[di] = 0;
  else ((uint16_t*)dst)[di] = 0; /* +0 */
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------------------- */
/* prune  (Section 3 pattern; Section 4.1 step 2)                                        */
/* ------------------------------------------------------------------------------------- */
void oracle_prune(int dtype, int64_t M, int64_t K, const void* x, int64_t ldx, void* y,
                  int64_t ldy) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t g = 0; g < K / 4; ++g) {
      int key[4], p0, p1;
      for (int p = 0; p < 4; ++p) key[p] = magnitude_key(dtype, x, i * ldx + 4 * g + p);
      select_two(key, &p0, &p1);
      for (int p = 0; p < 4; ++p) {
        if (p == p0 || p == p1) copy_elem(dtype, y, i * ldy + 4 * g + p, x, i * ldx + 4 * g + p);
        else zero_elem(dtype, y, i * ldy + 4 * g + p);
      }
    }
  }
}

/* ------------------------------------------------------------------------------------- */
/* compress  (Section 3.1, Figure 1)                                                      */
/* vals is M x K/2; meta is the canonical layout: K/8 bytes per row, group g in bits       */
/* 4g..4g+3 of the row's little-endian bit string, nibble = p0 | p1 << 2.                  */
/* Returns the number of dropped positions whose magnitude was non-zero.                   */
/* ------------------------------------------------------------------------------------- */
int64_t oracle_compress(int dtype, int64_t M, int64_t K, const void* x, int64_t ldx, void* vals,
                        int64_t ldv, uint8_t* meta) {
  int64_t dropped = 0;
  memset(meta, 0, (size_t)(M * (K / 8)));
#pragma omp parallel for schedule(static) reduction(+ : dropped)
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t g = 0; g < K / 4; ++g) {
      int key[4], p0, p1;
      for (int p = 0; p < 4; ++p) key[p] = magnitude_key(dtype, x, i * ldx + 4 * g + p);
      select_two(key, &p0, &p1);
      copy_elem(dtype, vals, i * ldv + 2 * g, x, i * ldx + 4 * g + p0);
      copy_elem(dtype, vals, i * ldv + 2 * g + 1, x, i * ldx + 4 * g + p1);
      uint8_t nibble = (uint8_t)(p0 | (p1 << 2));
      meta[i * (K / 8) + g / 2] |= (uint8_t)(nibble << (4 * (g % 2)));
      for (int p = 0; p < 4; ++p)
        if (p != p0 && p != p1 && key[p] != 0) ++dropped;
    }
  }
  return dropped;
}

static void nibble_positions(const uint8_t* meta, int64_t K, int64_t i, int64_t g, int* p0,
                             int* p1) {
  uint8_t byte = meta[i * (K / 8) + g / 2];
  int nibble = (byte >> (4 * (g % 2))) & 0xF;
  *p0 = nibble & 3;
  *p1 = (nibble >> 2) & 3;
}

/* ------------------------------------------------------------------------------------- */
/* decompress: the metadata decodes the compressed format (Section 3.1)                   */
/* ------------------------------------------------------------------------------------- */
void oracle_decompress(int dtype, int64_t M, int64_t K, const void* vals, int64_t ldv,
                       const uint8_t* meta, void* y, int64_t ldy) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t k = 0; k < K; ++k) zero_elem(dtype, y, i * ldy + k);
    for (int64_t g = 0; g < K / 4; ++g) {
      int p0, p1;
      nibble_positions(meta, K, i, g, &p0, &p1);
      copy_elem(dtype, y, i * ldy + 4 * g + p0, vals, i * ldv + 2 * g);
      copy_elem(dtype, y, i * ldy + 4 * g + p1, vals, i * ldv + 2 * g + 1);
    }
  }
}

/* ------------------------------------------------------------------------------------- */
/* Tensor-core operand order of the metadata.                                             */
/* The nibbles of the canonical layout, permuted into 2048-byte blocks that each cover     */
/* 128 rows x 128 columns of A.  Rows are padded to a multiple of 128 and K to a multiple  */
/* of 256; padding nibbles are 0x4 (positions 0,1).  Block (mb, kb) starts at byte         */
/* (mb * KB + kb) * 2048 with KB = 2 * ceil(K / 256).  Inside a block, for local row r,    */
/* local group q (0..31):                                                                  */
/*   int8:  bit = 128*r + 4*q                                                              */
/*   16-bit types: rows are paired (r, r+8) inside each 16-row band and the two 16-column  */
/*          halves of every 32-column slice are split across lanes:                        */
/*          bit = 128*(r%8) + 16*((r/8)%2) + 2048*(r/16)                                   */
/*              + 1024*((q/4)%2) + 32*(q/8) + 4*(q%4)                                      */
/* direction 0: canonical -> operand order, 1: operand order -> canonical.                 */
/* ------------------------------------------------------------------------------------- */
static int64_t operand_bit_in_block(int dtype, int r, int q) {
  if (elem_size(dtype) == 1) return 128 * (int64_t)r + 4 * q;
  return 128 * (r % 8) + 16 * ((r / 8) % 2) + 2048 * (r / 16) + 1024 * ((q / 4) % 2) +
         32 * (q / 8) + 4 * (q % 4);
}

int64_t oracle_meta_operand_bytes(int64_t M, int64_t K) {
  int64_t MB = (M + 127) / 128, KB = 2 * ((K + 255) / 256);
  return MB * KB * 2048;
}

void oracle_meta_permute(int dtype, int64_t M, int64_t K, const uint8_t* src, uint8_t* dst,
                         int direction) {
  int64_t MB = (M + 127) / 128, KB = 2 * ((K + 255) / 256);
  if (direction == 0) memset(dst, 0x44, (size_t)(MB * KB * 2048));
  else memset(dst, 0, (size_t)(M * (K / 8)));
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t g = 0; g < K / 4; ++g) {
      int64_t mb = i / 128, kb = g / 32;
      int r = (int)(i % 128), q = (int)(g % 32);
      int64_t bit = ((mb * KB + kb) * 2048) * 8 + operand_bit_in_block(dtype, r, q);
      int64_t cbyte = i * (K / 8) + g / 2;
      int cshift = 4 * (int)(g % 2);
      int64_t obyte = bit / 8;
      int oshift = (int)(bit % 8);
      if (direction == 0) {
        int nibble = (src[cbyte] >> cshift) & 0xF;
        dst[obyte] = (uint8_t)((dst[obyte] & ~(0xF << oshift)) | (nibble << oshift));
      } else {
        int nibble = (src[obyte] >> oshift) & 0xF;
        dst[cbyte] |= (uint8_t)(nibble << cshift);
      }
    }
  }
}

/* ------------------------------------------------------------------------------------- */
/* GEMM  (Section 3.2, Figure 2)                                                           */
/* D[i,j] = alpha * sum_g sum_t vals[i,2g+t] * B[4g+p_t(i,g), j] + beta * C[i,j]           */
/* on the output window rows [i0,i1) x columns [j0,j1); out is (i1-i0) x (j1-j0) packed.   */
/* B element (k, j) is B[k + j*ldb] when b_k_contiguous, else B[k*ldb + j].                */
/* C element (i, j) is C[i*ldc + j]; c_dtype codes: 0 fp16, 1 bf16, 3 fp32, 4 int32.       */
/* Floating point: out_f64 receives the un-rounded double result.                          */
/* int8: exact int64 accumulation, out_i32 receives the value cast to int32.               */
/* ------------------------------------------------------------------------------------- */
static double load_c(int c_dtype, const void* C, int64_t index) {
  if (c_dtype == 0) return half_bits_to_double(((const uint16_t*)C)[index]);
  if (c_dtype == 1) return bf16_bits_to_double(((const uint16_t*)C)[index]);
  if (c_dtype == 3) return (double)((const float*)C)[index];
  return (double)((const int32_t*)C)[index];
}

void oracle_gemm_sparse(int dtype, int64_t M, int64_t N, int64_t K, const void* vals,
                        int64_t ldv, const uint8_t* meta, const void* B, int64_t ldb,
                        int b_k_contiguous, double alpha, double beta, int c_dtype,
                        const void* C, int64_t ldc, int64_t i0, int64_t i1, int64_t j0,
                        int64_t j1, double* out_f64, int32_t* out_i32) {
  (void)M;
  (void)N;
  int64_t width = j1 - j0;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t i = i0; i < i1; ++i) {
    for (int64_t j = j0; j < j1; ++j) {
      double acc = 0.0;
      int64_t iacc = 0;
      for (int64_t g = 0; g < K / 4; ++g) {
        int p[2];
        nibble_positions(meta, K, i, g, &p[0], &p[1]);
        for (int t = 0; t < 2; ++t) {
          int64_t k = 4 * g + p[t];
          int64_t bidx = b_k_contiguous ? k + j * ldb : k * ldb + j;
          if (dtype == 2) {
            iacc += (int64_t)((const int8_t*)vals)[i * ldv + 2 * g + t] *
                    (int64_t)((const int8_t*)B)[bidx];
          } else {
            acc += load_as_double(dtype, vals, i * ldv + 2 * g + t) * load_as_double(dtype, B, bidx);
          }
        }
      }
      int64_t o = (i - i0) * width + (j - j0);
      if (dtype == 2) {
        int64_t r = (int64_t)alpha * iacc;
        if (beta != 0.0 && C) r += (int64_t)beta * (int64_t)((const int32_t*)C)[i * ldc + j];
        out_i32[o] = (int32_t)r;
      } else {
        double r = alpha * acc;
        if (beta != 0.0 && C) r += beta * load_c(c_dtype, C, i * ldc + j);
        out_f64[o] = r;
      }
    }
  }
}

/* The textbook dense product on a dense A (used on prune(x) and on decompress(...)):
 * D[i,j] = alpha * sum_k A[i,k] * B[k,j] + beta * C[i,j], k ascending. */
void oracle_gemm_dense(int dtype, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                       const void* B, int64_t ldb, int b_k_contiguous, double alpha, double beta,
                       int c_dtype, const void* C, int64_t ldc, int64_t i0, int64_t i1,
                       int64_t j0, int64_t j1, double* out_f64, int32_t* out_i32) {
  (void)M;
  (void)N;
  int64_t width = j1 - j0;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t i = i0; i < i1; ++i) {
    for (int64_t j = j0; j < j1; ++j) {
      double acc = 0.0;
      int64_t iacc = 0;
      for (int64_t k = 0; k < K; ++k) {
        int64_t bidx = b_k_contiguous ? k + j * ldb : k * ldb + j;
        if (dtype == 2) {
          iacc += (int64_t)((const int8_t*)A)[i * lda + k] * (int64_t)((const int8_t*)B)[bidx];
        } else {
          acc += load_as_double(dtype, A, i * lda + k) * load_as_double(dtype, B, bidx);
        }
      }
      int64_t o = (i - i0) * width + (j - j0);
      if (dtype == 2) {
        int64_t r = (int64_t)alpha * iacc;
        if (beta != 0.0 && C) r += (int64_t)beta * (int64_t)((const int32_t*)C)[i * ldc + j];
        out_i32[o] = (int32_t)r;
      } else {
        double r = alpha * acc;
        if (beta != 0.0 && C) r += beta * load_c(c_dtype, C, i * ldc + j);
        out_f64[o] = r;
      }
    }
  }
}

/* sum_k |A[i,k]| * |B[k,j]| over the kept values, in double: the scale of the per-element
 * error bound for the floating-point GEMM. */
void oracle_gemm_abs(int dtype, int64_t K, const void* vals, int64_t ldv, const uint8_t* meta,
                     const void* B, int64_t ldb, int b_k_contiguous, int64_t i0, int64_t i1,
                     int64_t j0, int64_t j1, double* out_f64) {
  int64_t width = j1 - j0;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t i = i0; i < i1; ++i) {
    for (int64_t j = j0; j < j1; ++j) {
      double acc = 0.0;
      for (int64_t g = 0; g < K / 4; ++g) {
        int p[2];
        nibble_positions(meta, K, i, g, &p[0], &p[1]);
        for (int t = 0; t < 2; ++t) {
          int64_t k = 4 * g + p[t];
          int64_t bidx = b_k_contiguous ? k + j * ldb : k * ldb + j;
          acc += fabs(load_as_double(dtype, vals, i * ldv + 2 * g + t)) *
                 fabs(load_as_double(dtype, B, bidx));
        }
      }
      out_f64[(i - i0) * width + (j - j0)] = acc;
    }
  }
}

/* ------------------------------------------------------------------------------------- */
/* im2col for a 3x3, stride 1, pad 1 convolution on NHWC input (Section 4.2: the           */
/* reduction dimension of a convolution is C*R*S).  K index = (r*3 + s)*C + c, output      */
/* column = (n*H + h)*W + w, stored K-contiguous with leading dimension ldo.               */
/* ------------------------------------------------------------------------------------- */
void oracle_im2col_nhwc_3x3(int dtype, int64_t Nb, int64_t H, int64_t W, int64_t C,
                            const void* in, void* out, int64_t ldo) {
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < Nb; ++n)
    for (int64_t h = 0; h < H; ++h)
      for (int64_t w = 0; w < W; ++w)
        for (int r = 0; r < 3; ++r)
          for (int s = 0; s < 3; ++s)
            for (int64_t c = 0; c < C; ++c) {
              int64_t hh = h + r - 1, ww = w + s - 1;
              int64_t o = ((n * H + h) * W + w) * ldo + (r * 3 + s) * C + c;
              if (hh < 0 || hh >= H || ww < 0 || ww >= W) zero_elem(dtype, out, o);
              else copy_elem(dtype, out, o, in, ((n * H + hh) * W + ww) * C + c);
            }
}

/* ------------------------------------------------------------------------------------- */
/* The 1:2 pattern of the TF32 mode (Section 3.2: with FP32 input/output the pattern becomes */
/* 1:2, i.e. one kept value in every aligned pair; Table 1, TF32 row).                        */
/* FP32 storage as bit patterns (uint32).  Selection: larger magnitude (bit pattern without  */
/* the sign), equal magnitudes keep the lower index.  Compressed form: vals M x K/2 and one  */
/* nibble per pair, 0x4 if the first element is kept, 0xE if the second: the pair seen as    */
/* four 16-bit halves of which halves (0,1) or (2,3) are kept, the 2:4 code of Section 3.1.  */
/* Canonical layout: pair g of row i in bits 4g..4g+3 of the row (K/4 bytes per row).        */
/* ------------------------------------------------------------------------------------- */
static int keep_second_of_pair(const uint32_t* x, int64_t idx) {
  uint32_t k0 = x[idx] & 0x7FFFFFFFu, k1 = x[idx + 1] & 0x7FFFFFFFu;
  return k1 > k0; /* tie -> first */
}

void oracle_prune_1of2(int64_t M, int64_t K, const uint32_t* x, int64_t ldx, uint32_t* y, int64_t ldy) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t g = 0; g < K / 2; ++g) {
      int second = keep_second_of_pair(x, i * ldx + 2 * g);
      y[i * ldy + 2 * g] = second ? 0u : x[i * ldx + 2 * g];
      y[i * ldy + 2 * g + 1] = second ? x[i * ldx + 2 * g + 1] : 0u;
    }
}

int64_t oracle_compress_1of2(int64_t M, int64_t K, const uint32_t* x, int64_t ldx, uint32_t* vals, int64_t ldv,
                             uint8_t* meta) {
  int64_t dropped = 0;
  memset(meta, 0, (size_t)(M * (K / 4)));
  for (int64_t i = 0; i < M; ++i)
    for (int64_t g = 0; g < K / 2; ++g) {
      int second = keep_second_of_pair(x, i * ldx + 2 * g);
      vals[i * ldv + g] = x[i * ldx + 2 * g + second];
      uint8_t nibble = second ? 0xE : 0x4;
      meta[i * (K / 4) + g / 2] |= (uint8_t)(nibble << (4 * (g % 2)));
      if ((x[i * ldx + 2 * g + (1 - second)] & 0x7FFFFFFFu) != 0) ++dropped;
    }
  return dropped;
}

static int pair_kept_index(const uint8_t* meta, int64_t K, int64_t i, int64_t g) {
  int nibble = (meta[i * (K / 4) + g / 2] >> (4 * (g % 2))) & 0xF;
  return (nibble & 3) >> 1; /* halves (0,1) -> element 0, halves (2,3) -> element 1 */
}

void oracle_decompress_1of2(int64_t M, int64_t K, const uint32_t* vals, int64_t ldv, const uint8_t* meta, uint32_t* y,
                            int64_t ldy) {
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t k = 0; k < K; ++k) y[i * ldy + k] = 0u;
    for (int64_t g = 0; g < K / 2; ++g) y[i * ldy + 2 * g + pair_kept_index(meta, K, i, g)] = vals[i * ldv + g];
  }
}

static double f32_bits_to_double(uint32_t w) {
  float f;
  memcpy(&f, &w, sizeof f);
  return (double)f;
}

/* D[i,j] = alpha * sum_g vals[i,g] * B[2g + e(i,g), j] + beta * C[i,j], doubles throughout; B as   */
/* N rows of K values (K contiguous); C fp32 (row-major, ldc); out_abs receives sum |a||b|.         */
void oracle_gemm_sparse_1of2(int64_t K, const uint32_t* vals, int64_t ldv, const uint8_t* meta, const uint32_t* Bt,
                             int64_t ldb, double alpha, double beta, const float* C, int64_t ldc, int64_t i0,
                             int64_t i1, int64_t j0, int64_t j1, double* out, double* out_abs) {
  int64_t width = j1 - j0;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t i = i0; i < i1; ++i)
    for (int64_t j = j0; j < j1; ++j) {
      double acc = 0.0, mag = 0.0;
      for (int64_t g = 0; g < K / 2; ++g) {
        int64_t k = 2 * g + pair_kept_index(meta, K, i, g);
        double a = f32_bits_to_double(vals[i * ldv + g]), b = f32_bits_to_double(Bt[j * ldb + k]);
        acc += a * b;
        mag += fabs(a) * fabs(b);
      }
      double r = alpha * acc;
      if (beta != 0.0 && C) r += beta * (double)C[i * ldc + j];
      out[(i - i0) * width + (j - j0)] = r;
      if (out_abs) out_abs[(i - i0) * width + (j - j0)] = mag;
    }
}

/* Operand order of the 1:2 metadata: the same nibble placement as the 16-bit types (a block  */
/* is 128 rows x 32 nibbles), but a nibble stands for a pair, so a block covers 64 columns    */
/* and K is padded to a multiple of 128.                                                      */
int64_t oracle_meta_operand_bytes_1of2(int64_t M, int64_t K) {
  return ((M + 127) / 128) * (2 * ((K + 127) / 128)) * 2048;
}

void oracle_meta_permute_1of2(int64_t M, int64_t K, const uint8_t* src, uint8_t* dst, int direction) {
  int64_t MB = (M + 127) / 128, KB = 2 * ((K + 127) / 128);
  if (direction == 0) memset(dst, 0x44, (size_t)(MB * KB * 2048));
  else memset(dst, 0, (size_t)(M * (K / 4)));
  for (int64_t i = 0; i < M; ++i)
    for (int64_t g = 0; g < K / 2; ++g) {
      int64_t mb = i / 128, kb = g / 32;
      int r = (int)(i % 128), q = (int)(g % 32);
      int64_t bit = ((mb * KB + kb) * 2048) * 8 + operand_bit_in_block(0, r, q);
      int64_t cbyte = i * (K / 4) + g / 2, obyte = bit / 8;
      int cshift = 4 * (int)(g % 2), oshift = (int)(bit % 8);
      if (direction == 0) {
        int nibble = (src[cbyte] >> cshift) & 0xF;
        dst[obyte] = (uint8_t)((dst[obyte] & ~(0xF << oshift)) | (nibble << oshift));
      } else {
        dst[cbyte] |= (uint8_t)(((src[obyte] >> oshift) & 0xF) << cshift);
      }
    }
}

/* ------------------------------------------------------------------------------------- */
/* Dequantising epilogue of the INT8 deployment (Section 4.4; Section 5.1: per-row scaling  */
/* factors for fully-connected weights, a per-tensor factor for activations).  acc is the    */
/* exact INT32 product; row_scale[i] already contains the activation factor.                */
/*   out_f64:  y = row_scale[i] * acc + bias[i] in double, then the activation.             */
/*   out_i8 :  the quantised code.  A rounding decision has to be taken in one precision on */
/*             both sides, and the method fixes none, so it is the kernel's: float(acc)     */
/*             (round to nearest), one fused multiply-add, the activation, one multiply by  */
/*             1/out_scale (itself rounded to float), round-half-to-even, clamp to +-127.   */
/* ------------------------------------------------------------------------------------- */
void oracle_dequant(int64_t rows, int64_t cols, const int32_t* acc, const float* row_scale,
                    const float* bias, int relu, float out_scale, double* out_f64, int8_t* out_i8) {
  const float inv = 1.0f / out_scale;
  for (int64_t i = 0; i < rows; ++i) {
    for (int64_t j = 0; j < cols; ++j) {
      int32_t a = acc[i * cols + j];
      float b = bias ? bias[i] : 0.0f;
      if (out_f64) {
        double y = (double)row_scale[i] * (double)a + (double)b;
        if (relu && y < 0.0) y = 0.0;
        out_f64[i * cols + j] = y;
      }
      if (out_i8) {
        float t = (float)a;
        float y = fmaf(row_scale[i], t, b);
        if (relu && !(y > 0.0f)) y = 0.0f;
        volatile float z = y * inv; /* volatile: one rounding to float, no wider intermediate */
        float q = rintf(z);
        if (q > 127.0f) q = 127.0f;
        if (q < -127.0f) q = -127.0f;
        out_i8[i * cols + j] = (int8_t)q;
      }
    }
  }
}

/* ------------------------------------------------------------------------------------- */
/* Tools around the pruning step.                                                          */
/* ------------------------------------------------------------------------------------- */
/* Section 4.1 (channel permutations): total magnitude kept by 2:4 pruning of the matrix    */
/* whose column k is column perm[k] of x (perm NULL = identity), summed in double.          */
double oracle_kept_magnitude(int dtype, int64_t M, int64_t K, const void* x, int64_t ldx, const int32_t* perm) {
  double total = 0.0;
  for (int64_t i = 0; i < M; ++i)
    for (int64_t g = 0; g < K / 4; ++g) {
      int key[4], p0, p1;
      int64_t idx[4];
      for (int p = 0; p < 4; ++p) {
        idx[p] = i * ldx + (perm ? perm[4 * g + p] : 4 * g + p);
        key[p] = magnitude_key(dtype, x, idx[p]);
      }
      select_two(key, &p0, &p1);
      total += fabs(load_as_double(dtype, x, idx[p0])) + fabs(load_as_double(dtype, x, idx[p1]));
    }
  return total;
}

/* Section 4.1 step 3: the pattern stays fixed while the weights change: keep w where the    */
/* canonical metadata names the position, +0 elsewhere.                                       */
void oracle_apply_mask(int dtype, int64_t M, int64_t K, const void* w, int64_t ldw, const uint8_t* meta, void* y,
                       int64_t ldy) {
  for (int64_t i = 0; i < M; ++i)
    for (int64_t g = 0; g < K / 4; ++g) {
      int p0, p1;
      nibble_positions(meta, K, i, g, &p0, &p1);
      for (int p = 0; p < 4; ++p) {
        if (p == p0 || p == p1) copy_elem(dtype, y, i * ldy + 4 * g + p, w, i * ldw + 4 * g + p);
        else zero_elem(dtype, y, i * ldy + 4 * g + p);
      }
    }
}

/* Section 6: 2:4 along rows and columns of every aligned 4 x 4 block.  All assignments of one of  */
/* the six pairs {01,02,03,12,13,23} to each of the four rows are visited in lexicographic order;  */
/* those whose columns all hold exactly two kept entries are the 90 candidates.  Which one is      */
/* "largest" is a floating-point decision and the method fixes no precision, so it is the kernel's: */
/* score = ((s0 + s1) + s2) + s3, s_i = |x[i,c]| + |x[i,c']|, all in float; the first candidate    */
/* with the strictly largest score wins.                                                           */
void oracle_prune_2d(int dtype, int64_t M, int64_t K, const void* x, int64_t ldx, void* y, int64_t ldy) {
  static const int pair[6][2] = {{0, 1}, {0, 2}, {0, 3}, {1, 2}, {1, 3}, {2, 3}};
  for (int64_t bi = 0; bi < M / 4; ++bi)
    for (int64_t bj = 0; bj < K / 4; ++bj) {
      float mag[4][4];
      for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j) mag[i][j] = (float)fabs(load_as_double(dtype, x, (4 * bi + i) * ldx + 4 * bj + j));
      float best = -1.0f;
      int best_rows[4] = {0, 0, 0, 0};
      int r[4];
      for (r[0] = 0; r[0] < 6; ++r[0])
        for (r[1] = 0; r[1] < 6; ++r[1])
          for (r[2] = 0; r[2] < 6; ++r[2])
            for (r[3] = 0; r[3] < 6; ++r[3]) {
              int col[4] = {0, 0, 0, 0};
              for (int i = 0; i < 4; ++i) { ++col[pair[r[i]][0]]; ++col[pair[r[i]][1]]; }
              if (col[0] != 2 || col[1] != 2 || col[2] != 2 || col[3] != 2) continue;
              volatile float sc = 0.0f;
              for (int i = 0; i < 4; ++i) {
                volatile float si = mag[i][pair[r[i]][0]] + mag[i][pair[r[i]][1]];
                sc = (i == 0) ? si : sc + si;
              }
              if (sc > best) { best = sc; for (int i = 0; i < 4; ++i) best_rows[i] = r[i]; }
            }
      for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j) {
          int keep = j == pair[best_rows[i]][0] || j == pair[best_rows[i]][1];
          if (keep) copy_elem(dtype, y, (4 * bi + i) * ldy + 4 * bj + j, x, (4 * bi + i) * ldx + 4 * bj + j);
          else zero_elem(dtype, y, (4 * bi + i) * ldy + 4 * bj + j);
        }
    }
}

int oracle_elem_size(int dtype) { return elem_size(dtype); }

/* Exact widening of n stored elements to double. */
void oracle_to_double(int dtype, int64_t n, const void* x, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = load_as_double(dtype, x, i);
}
