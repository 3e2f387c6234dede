// Tools around the pruning step of the workflow (Section 4.1 and Section 6 of arXiv 2104.08378):
//   sp24_kept_magnitude  total magnitude that 2:4 pruning keeps, optionally under a column
//                        permutation: the figure of merit of the channel permutations of Section 4.1;
//   sp24_apply_mask      re-imposes a fixed 2:4 pattern (given as metadata) on changed weights: what
//                        sparse retraining (step 3) does after every update;
//   sp24_prune_2d        2:4 along rows AND columns of every 4x4 block, so that the transposed matrix
//                        is 2:4 as well (Section 6), by exhaustive search over the 90 such patterns.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "sp24_common.cuh"

namespace sp24 {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint32_t keep_mask4(uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3) {
  uint32_t c01 = k0 >= k1, c02 = k0 >= k2, c03 = k0 >= k3;
  uint32_t c12 = k1 >= k2, c13 = k1 >= k3, c23 = k2 >= k3;
  uint32_t b0 = 3u - (c01 + c02 + c03), b1 = c01 + 2u - (c12 + c13);
  uint32_t b2 = c02 + c12 + 1u - c23, b3 = c03 + c13 + c23;
  return (b0 < 2u) | ((b1 < 2u) << 1) | ((b2 < 2u) << 2) | ((b3 < 2u) << 3);
}

template <typename T>
__device__ __forceinline__ uint32_t key_of(T e) {
  return sizeof(T) == 2 ? (uint32_t)((uint16_t)e & 0x7FFFu) : (uint32_t)abs((int)(int8_t)e);
}

// |value| as a float, exact for all three storage types.  DT: 0 fp16, 1 bf16, 2 int8.
template <int DT, typename T>
__device__ __forceinline__ float magnitude_of(T e) {
  if (DT == 2) return (float)abs((int)(int8_t)e);
  uint16_t bits = (uint16_t)e & 0x7FFFu;
  if (DT == 0) return __half2float(*reinterpret_cast<__half*>(&bits));
  return __bfloat162float(*reinterpret_cast<__nv_bfloat16*>(&bits));
}

// ---- kept magnitude -------------------------------------------------------------------------------
template <int DT, typename T>
__global__ void __launch_bounds__(kThreads) kept_magnitude_kernel(const T* __restrict__ x, int64_t ldx, int64_t M,
                                                                  int64_t groups, const int32_t* __restrict__ perm,
                                                                  double* result) {
  double sum = 0.0;
  const int64_t total = M * groups;
  for (int64_t id = (int64_t)blockIdx.x * kThreads + threadIdx.x; id < total; id += (int64_t)gridDim.x * kThreads) {
    const int64_t row = id / groups, g = id - row * groups;
    T e[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int64_t col = perm ? (int64_t)perm[4 * g + p] : 4 * g + p;
      e[p] = x[row * ldx + col];
    }
    const uint32_t m = keep_mask4(key_of(e[0]), key_of(e[1]), key_of(e[2]), key_of(e[3]));
#pragma unroll
    for (int p = 0; p < 4; ++p)
      if ((m >> p) & 1u) sum += (double)magnitude_of<DT>(e[p]);
  }
  // block reduction, one atomic per block
  __shared__ double part[kThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) s += part[w];
    atomicAdd(result, s);
  }
}

// ---- apply mask -----------------------------------------------------------------------------------
// One thread per 8 columns (two groups = one metadata byte in either layout).
template <typename T>
__global__ void __launch_bounds__(kThreads) apply_mask_kernel(const T* __restrict__ w, int64_t ldw, const uint8_t* meta,
                                                              int layout, T* y, int64_t ldy, int64_t M, int64_t K,
                                                              int64_t KB) {
  constexpr int ES = sizeof(T);
  const int64_t bytes = K >> 3;
  const int64_t id = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (id >= M * bytes) return;
  const int64_t row = id / bytes, bi = id - row * bytes;
  int64_t off;
  if (layout == SP24_META_CANONICAL) {
    off = row * bytes + bi;
  } else {
    const int64_t chunk = bi >> 1, blk = (row >> 7) * KB + (chunk >> 3);
    const int r = (int)(row & 127), cl = (int)(chunk & 7);
    const int in_blk = ES == 2 ? 16 * (r & 7) + 2 * ((r >> 3) & 1) + 256 * (r >> 4) + 128 * (cl & 1) + 4 * (cl >> 1)
                               : 16 * r + 2 * cl;
    off = blk * 2048 + in_blk + (bi & 1);
  }
  const uint32_t mbyte = meta[off];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t nib = (mbyte >> (4 * h)) & 0xFu, p0 = nib & 3u, p1 = nib >> 2;
    const T* src = w + row * ldw + 8 * bi + 4 * h;
    T* dst = y + row * ldy + 8 * bi + 4 * h;
    T e[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) e[p] = src[p];
#pragma unroll
    for (int p = 0; p < 4; ++p) dst[p] = ((uint32_t)p == p0 || (uint32_t)p == p1) ? e[p] : (T)0;
  }
}

// ---- 2:4 along rows and columns ------------------------------------------------------------------------
// The 90 patterns: every row keeps one of the six pairs {01,02,03,12,13,23} (in that order, index 0..5)
// and every column ends up with exactly two kept entries.  Patterns are numbered in lexicographic order
// of their four row indices; kPatterns[n] packs the four 3-bit row indices of pattern n.
__constant__ uint16_t kPatterns[90];
__constant__ uint8_t kPairMask[6] = {0x3, 0x5, 0x9, 0x6, 0xA, 0xC};

// Score of a pattern: ((s0 + s1) + s2) + s3 with s_i = |x[i, c]| + |x[i, c']| (c < c'), all in FP32 (int32
// for int8); the first pattern with the largest score wins.
template <int DT, typename T>
__global__ void __launch_bounds__(kThreads) prune_2d_kernel(const T* __restrict__ x, int64_t ldx, T* y, int64_t ldy,
                                                            int64_t block_rows, int64_t block_cols) {
  const int64_t id = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (id >= block_rows * block_cols) return;
  const int64_t br = id / block_cols, bc = id - br * block_cols;
  T e[4][4];
  float s[4][6];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      e[i][j] = x[(4 * br + i) * ldx + 4 * bc + j];
      a[j] = magnitude_of<DT>(e[i][j]);
    }
    s[i][0] = __fadd_rn(a[0], a[1]); s[i][1] = __fadd_rn(a[0], a[2]); s[i][2] = __fadd_rn(a[0], a[3]);
    s[i][3] = __fadd_rn(a[1], a[2]); s[i][4] = __fadd_rn(a[1], a[3]); s[i][5] = __fadd_rn(a[2], a[3]);
  }
  float best = -1.f;
  uint32_t best_pat = 0;
  for (int n = 0; n < 90; ++n) {
    const uint32_t pat = kPatterns[n];
    float sc = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t idx = (pat >> (3 * i)) & 7u;
      float si = s[i][0];
#pragma unroll
      for (int q = 1; q < 6; ++q) si = idx == (uint32_t)q ? s[i][q] : si;
      sc = i == 0 ? si : __fadd_rn(sc, si);
    }
    if (sc > best) { best = sc; best_pat = pat; }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t m = kPairMask[(best_pat >> (3 * i)) & 7u];
#pragma unroll
    for (int j = 0; j < 4; ++j) y[(4 * br + i) * ldy + 4 * bc + j] = ((m >> j) & 1u) ? e[i][j] : (T)0;
  }
}

// Fills the pattern table once per device.
sp24_status upload_patterns() {
  static bool done[64] = {};
  int dev = 0;
  SP24_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && done[dev]) return SP24_OK;
  static const uint8_t pair_mask[6] = {0x3, 0x5, 0x9, 0x6, 0xA, 0xC};
  uint16_t table[90];
  int n = 0;
  for (int a = 0; a < 6; ++a)
    for (int b = 0; b < 6; ++b)
      for (int c = 0; c < 6; ++c)
        for (int d = 0; d < 6; ++d) {
          bool ok = true;
          for (int col = 0; col < 4; ++col) {
            int cnt = ((pair_mask[a] >> col) & 1) + ((pair_mask[b] >> col) & 1) + ((pair_mask[c] >> col) & 1) +
                      ((pair_mask[d] >> col) & 1);
            ok = ok && cnt == 2;
          }
          if (ok && n < 90) table[n++] = (uint16_t)(a | (b << 3) | (c << 6) | (d << 9));
        }
  if (n != 90) return SP24_ERR_CUDA;
  SP24_CUDA_CHECK(cudaMemcpyToSymbol(kPatterns, table, sizeof(table)));
  if (dev >= 0 && dev < 64) done[dev] = true;
  return SP24_OK;
}

}  // namespace
}  // namespace sp24

using namespace sp24;

extern "C" sp24_status sp24_kept_magnitude(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx,
                                           const int32_t* perm, double* result, void* stream) {
  SP24_RETURN_IF(!is_ab_type(t) || is_fp8(t), SP24_ERR_DTYPE);
  SP24_RETURN_IF(M < 0 || K < 0 || K % 4 != 0, SP24_ERR_SHAPE);
  SP24_RETURN_IF(result == nullptr, SP24_ERR_NULL);
  if (M == 0 || K == 0) return SP24_OK;
  SP24_RETURN_IF(x == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ldx < K, SP24_ERR_STRIDE);
  sp24_status st = check_arch();
  if (st != SP24_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t groups = K / 4, total = M * groups;
  int64_t blocks = (total + kThreads - 1) / kThreads;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (t == SP24_F16)
    kept_magnitude_kernel<0, uint16_t><<<(unsigned)blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, M, groups, perm, result);
  else if (t == SP24_BF16)
    kept_magnitude_kernel<1, uint16_t><<<(unsigned)blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, M, groups, perm, result);
  else
    kept_magnitude_kernel<2, int8_t><<<(unsigned)blocks, kThreads, 0, s>>>((const int8_t*)x, ldx, M, groups, perm, result);
  return cuda_status(cudaGetLastError());
}

extern "C" sp24_status sp24_apply_mask(sp24_dtype t, int64_t M, int64_t K, const void* w, int64_t ldw, const void* meta,
                                       sp24_meta_layout l, void* y, int64_t ldy, void* stream) {
  SP24_RETURN_IF(!is_ab_type(t), SP24_ERR_DTYPE);
  SP24_RETURN_IF(M < 0 || K < 0 || K % 8 != 0, SP24_ERR_SHAPE);
  SP24_RETURN_IF(l != SP24_META_CANONICAL && l != SP24_META_TCGEN05, SP24_ERR_UNSUPPORTED);
  if (M == 0 || K == 0) return SP24_OK;
  SP24_RETURN_IF(w == nullptr || meta == nullptr || y == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ldw < K || ldy < K, SP24_ERR_STRIDE);
  sp24_status st = check_arch();
  if (st != SP24_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t total = M * (K / 8), KB = 2 * ((K + 255) / 256);
  const unsigned blocks = (unsigned)((total + kThreads - 1) / kThreads);
  if (elem_bytes(t) == 2)
    apply_mask_kernel<uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)w, ldw, (const uint8_t*)meta, (int)l,
                                                            (uint16_t*)y, ldy, M, K, KB);
  else
    apply_mask_kernel<int8_t><<<blocks, kThreads, 0, s>>>((const int8_t*)w, ldw, (const uint8_t*)meta, (int)l, (int8_t*)y,
                                                          ldy, M, K, KB);
  return cuda_status(cudaGetLastError());
}

extern "C" sp24_status sp24_prune_2d(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx, void* y, int64_t ldy,
                                     void* stream) {
  SP24_RETURN_IF(!is_ab_type(t) || is_fp8(t), SP24_ERR_DTYPE);
  SP24_RETURN_IF(M < 0 || K < 0 || K % 4 != 0 || M % 4 != 0, SP24_ERR_SHAPE);
  if (M == 0 || K == 0) return SP24_OK;
  SP24_RETURN_IF(x == nullptr || y == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ldx < K || ldy < K, SP24_ERR_STRIDE);
  sp24_status st = check_arch();
  if (st != SP24_OK) return st;
  if ((st = upload_patterns()) != SP24_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t br = M / 4, bc = K / 4, total = br * bc;
  const unsigned blocks = (unsigned)((total + kThreads - 1) / kThreads);
  if (t == SP24_F16)
    prune_2d_kernel<0, uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, (uint16_t*)y, ldy, br, bc);
  else if (t == SP24_BF16)
    prune_2d_kernel<1, uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, (uint16_t*)y, ldy, br, bc);
  else
    prune_2d_kernel<2, int8_t><<<blocks, kThreads, 0, s>>>((const int8_t*)x, ldx, (int8_t*)y, ldy, br, bc);
  return cuda_status(cudaGetLastError());
}
