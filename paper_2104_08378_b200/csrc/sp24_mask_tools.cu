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
// One block sums its threads' partial sums and adds them to *result with one atomic.
__device__ __forceinline__ void block_add(double sum, double* result) {
  __shared__ double part[kThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
  const int t = threadIdx.x;
  if ((t & 31) == 0) part[t >> 5] = sum;
  __syncthreads();
  if (t == 0) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) s += part[w];
    atomicAdd(result, s);
  }
}

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
  block_add(sum, result);
}

// Kept magnitude of the groups held in one 16-byte vector (two groups of a 16-bit type, four of int8).
template <int DT>
__device__ __forceinline__ double kept_in_vector(uint4 v) {
  double sum = 0.0;
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  if (DT == 2) {
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t a = __vabs4(w[g]);  // -128 -> 128
      uint32_t k0 = a & 0xFFu, k1 = (a >> 8) & 0xFFu, k2 = (a >> 16) & 0xFFu, k3 = a >> 24;
      uint32_t m = keep_mask4(k0, k1, k2, k3);
      uint32_t kept = ((m & 1u) ? k0 : 0u) + ((m & 2u) ? k1 : 0u) + ((m & 4u) ? k2 : 0u) + ((m & 8u) ? k3 : 0u);
      sum += (double)kept;  // integers: exact
    }
  } else {
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      const uint32_t lo = w[2 * g] & 0x7FFF7FFFu, hi = w[2 * g + 1] & 0x7FFF7FFFu;
      const uint32_t k[4] = {lo & 0xFFFFu, lo >> 16, hi & 0xFFFFu, hi >> 16};
      const uint32_t m = keep_mask4(k[0], k[1], k[2], k[3]);
#pragma unroll
      for (int p = 0; p < 4; ++p)
        if ((m >> p) & 1u) sum += (double)magnitude_of<DT>((uint16_t)k[p]);
    }
  }
  return sum;
}

// Identity permutation, 16-byte aligned rows: threads along a row, one vector per thread and row step.
template <int DT>
__global__ void __launch_bounds__(kThreads) kept_magnitude_vec_kernel(const uint8_t* __restrict__ x, int64_t row_bytes,
                                                                      int64_t M, int64_t vpr, double* result) {
  double sum = 0.0;
  const int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (c < vpr) {
    for (int64_t row = blockIdx.y; row < M; row += gridDim.y)
      sum += kept_in_vector<DT>(__ldcs(reinterpret_cast<const uint4*>(x + row * row_bytes + c * 16)));
  }
  block_add(sum, result);
}

// Column permutation, 16-byte aligned rows of at most 48 KB: a block copies one row into shared memory
// with coalesced vector loads and gathers the permuted groups from there.
template <int DT, typename T>
__global__ void __launch_bounds__(kThreads) kept_magnitude_perm_kernel(const uint8_t* __restrict__ x, int64_t row_bytes,
                                                                       int64_t M, int64_t K,
                                                                       const int32_t* __restrict__ perm, double* result) {
  extern __shared__ uint4 row_buf[];
  const T* row_elems = reinterpret_cast<const T*>(row_buf);
  const int64_t vpr = K * (int64_t)sizeof(T) / 16, groups = K / 4;
  double sum = 0.0;
  for (int64_t row = blockIdx.x; row < M; row += gridDim.x) {
    for (int64_t c = threadIdx.x; c < vpr; c += kThreads)
      row_buf[c] = __ldcs(reinterpret_cast<const uint4*>(x + row * row_bytes + c * 16));
    __syncthreads();
    for (int64_t g = threadIdx.x; g < groups; g += kThreads) {
      const int4 pc = *reinterpret_cast<const int4*>(perm + 4 * g);
      T e[4] = {row_elems[pc.x], row_elems[pc.y], row_elems[pc.z], row_elems[pc.w]};
      const uint32_t m = keep_mask4(key_of(e[0]), key_of(e[1]), key_of(e[2]), key_of(e[3]));
#pragma unroll
      for (int p = 0; p < 4; ++p)
        if ((m >> p) & 1u) sum += (double)magnitude_of<DT>(e[p]);
    }
    __syncthreads();
  }
  block_add(sum, result);
}

// ---- apply mask -----------------------------------------------------------------------------------
// Vector path: one thread per 16 columns (four groups = 16 metadata bits), threads along a row.
template <int ES>
__global__ void __launch_bounds__(kThreads) apply_mask_vec_kernel(const uint8_t* w, int64_t row_bytes_w,
                                                                  const uint8_t* __restrict__ meta, int layout,
                                                                  uint8_t* y, int64_t row_bytes_y, int64_t M, int64_t K,
                                                                  int64_t KB) {
  const int64_t chunk = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (chunk >= (K >> 4)) return;
  const int cl = (int)(chunk & 7);
  for (int64_t row = blockIdx.y; row < M; row += gridDim.y) {
    int64_t off;
    if (layout == SP24_META_CANONICAL) {
      off = row * (K >> 3) + 2 * chunk;
    } else {
      const int r = (int)(row & 127);
      const int in_blk = ES == 2 ? 16 * (r & 7) + 2 * ((r >> 3) & 1) + 256 * (r >> 4) + 128 * (cl & 1) + 4 * (cl >> 1)
                                 : 16 * r + 2 * cl;
      off = ((row >> 7) * KB + (chunk >> 3)) * 2048 + in_blk;
    }
    const uint32_t mbits = *reinterpret_cast<const uint16_t*>(meta + off);
    if (ES == 2) {
      const uint8_t* src = w + row * row_bytes_w + chunk * 32;
      uint4 a = __ldcs(reinterpret_cast<const uint4*>(src)), b = __ldcs(reinterpret_cast<const uint4*>(src + 16));
      uint32_t v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t nib = (mbits >> (4 * g)) & 0xFu, keep = (1u << (nib & 3u)) | (1u << (nib >> 2));
        v[2 * g] &= ((keep & 1u) ? 0xFFFFu : 0u) | ((keep & 2u) ? 0xFFFF0000u : 0u);
        v[2 * g + 1] &= ((keep & 4u) ? 0xFFFFu : 0u) | ((keep & 8u) ? 0xFFFF0000u : 0u);
      }
      uint8_t* dst = y + row * row_bytes_y + chunk * 32;
      __stcs(reinterpret_cast<uint4*>(dst), make_uint4(v[0], v[1], v[2], v[3]));
      __stcs(reinterpret_cast<uint4*>(dst + 16), make_uint4(v[4], v[5], v[6], v[7]));
    } else {
      uint4 a = __ldcs(reinterpret_cast<const uint4*>(w + row * row_bytes_w + chunk * 16));
      uint32_t v[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t nib = (mbits >> (4 * g)) & 0xFu, keep = (1u << (nib & 3u)) | (1u << (nib >> 2));
        v[g] &= ((keep & 1u) ? 0xFFu : 0u) | ((keep & 2u) ? 0xFF00u : 0u) | ((keep & 4u) ? 0xFF0000u : 0u) |
                ((keep & 8u) ? 0xFF000000u : 0u);
      }
      __stcs(reinterpret_cast<uint4*>(y + row * row_bytes_y + chunk * 16), make_uint4(v[0], v[1], v[2], v[3]));
    }
  }
}


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
// of their four row indices; entry n packs the four 3-bit row indices of pattern n.  The table is built
// at compile time so that the search below unrolls into straight-line code on registers.
struct PatternTable {
  uint16_t v[90];
};
constexpr uint32_t pair_mask(int q) { return q == 0 ? 0x3u : q == 1 ? 0x5u : q == 2 ? 0x9u : q == 3 ? 0x6u : q == 4 ? 0xAu : 0xCu; }
constexpr PatternTable make_patterns() {
  PatternTable t{};
  int n = 0;
  for (int a = 0; a < 6; ++a)
    for (int b = 0; b < 6; ++b)
      for (int c = 0; c < 6; ++c)
        for (int d = 0; d < 6; ++d) {
          bool ok = true;
          for (int col = 0; col < 4; ++col) {
            const uint32_t cnt = ((pair_mask(a) >> col) & 1u) + ((pair_mask(b) >> col) & 1u) +
                                 ((pair_mask(c) >> col) & 1u) + ((pair_mask(d) >> col) & 1u);
            ok = ok && cnt == 2u;
          }
          if (ok && n < 90) t.v[n++] = (uint16_t)(a | (b << 3) | (c << 6) | (d << 9));
        }
  return t;
}
constexpr PatternTable kPatternTable = make_patterns();
static_assert(kPatternTable.v[89] != 0 && kPatternTable.v[0] == (0 | (0 << 3) | (5 << 6) | (5 << 9)),
              "90 patterns, the first keeps columns 0,1 in rows 0,1 and 2,3 in rows 2,3");

template <int N>
struct PatternSearch {
  // patterns N..89 in order; `s[i][q]`: kept magnitude of row i under pair q
  static __device__ __forceinline__ void run(const float (&s)[4][6], float& best, uint32_t& best_pat) {
    constexpr uint32_t pat = kPatternTable.v[N];
    const float sc = __fadd_rn(__fadd_rn(__fadd_rn(s[0][pat & 7u], s[1][(pat >> 3) & 7u]), s[2][(pat >> 6) & 7u]),
                               s[3][(pat >> 9) & 7u]);
    if (sc > best) { best = sc; best_pat = pat; }
    PatternSearch<N + 1>::run(s, best, best_pat);
  }
};
template <>
struct PatternSearch<90> {
  static __device__ __forceinline__ void run(const float (&)[4][6], float&, uint32_t&) {}
};

// Score of a pattern: ((s0 + s1) + s2) + s3 with s_i = |x[i, c]| + |x[i, c']| (c < c'), all in FP32 (exact
// for int8); the first pattern with the largest score wins.  One thread per 4 x 4 block.
template <int DT, typename T>
__global__ void __launch_bounds__(kThreads) prune_2d_kernel(const T* __restrict__ x, int64_t ldx, T* y, int64_t ldy,
                                                            int64_t block_rows, int64_t block_cols) {
  const int64_t bc = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (bc >= block_cols) return;
  for (int64_t br = blockIdx.y; br < block_rows; br += gridDim.y) {
    T e[4][4];
    float s[4][6];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const T* src = x + (4 * br + i) * ldx + 4 * bc;
      if (sizeof(T) == 2 && ((reinterpret_cast<uintptr_t>(src) & 7u) == 0)) {
        const uint2 v = *reinterpret_cast<const uint2*>(src);
        e[i][0] = (T)(v.x & 0xFFFFu); e[i][1] = (T)(v.x >> 16); e[i][2] = (T)(v.y & 0xFFFFu); e[i][3] = (T)(v.y >> 16);
      } else if (sizeof(T) == 1 && ((reinterpret_cast<uintptr_t>(src) & 3u) == 0)) {
        const uint32_t v = *reinterpret_cast<const uint32_t*>(src);
        e[i][0] = (T)(v & 0xFFu); e[i][1] = (T)((v >> 8) & 0xFFu); e[i][2] = (T)((v >> 16) & 0xFFu); e[i][3] = (T)(v >> 24);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) e[i][j] = src[j];
      }
      float a[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) a[j] = magnitude_of<DT>(e[i][j]);
      s[i][0] = __fadd_rn(a[0], a[1]); s[i][1] = __fadd_rn(a[0], a[2]); s[i][2] = __fadd_rn(a[0], a[3]);
      s[i][3] = __fadd_rn(a[1], a[2]); s[i][4] = __fadd_rn(a[1], a[3]); s[i][5] = __fadd_rn(a[2], a[3]);
    }
    float best = -1.f;
    uint32_t best_pat = 0;
    PatternSearch<0>::run(s, best, best_pat);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t q = (best_pat >> (3 * i)) & 7u;
      const uint32_t m = q == 0 ? 0x3u : q == 1 ? 0x5u : q == 2 ? 0x9u : q == 3 ? 0x6u : q == 4 ? 0xAu : 0xCu;
      T* dst = y + (4 * br + i) * ldy + 4 * bc;
      T o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) o[j] = ((m >> j) & 1u) ? e[i][j] : (T)0;
      if (sizeof(T) == 2 && ((reinterpret_cast<uintptr_t>(dst) & 7u) == 0)) {
        *reinterpret_cast<uint2*>(dst) = make_uint2((uint32_t)(uint16_t)o[0] | ((uint32_t)(uint16_t)o[1] << 16),
                                                     (uint32_t)(uint16_t)o[2] | ((uint32_t)(uint16_t)o[3] << 16));
      } else if (sizeof(T) == 1 && ((reinterpret_cast<uintptr_t>(dst) & 3u) == 0)) {
        *reinterpret_cast<uint32_t*>(dst) = (uint32_t)(uint8_t)o[0] | ((uint32_t)(uint8_t)o[1] << 8) |
                                            ((uint32_t)(uint8_t)o[2] << 16) | ((uint32_t)(uint8_t)o[3] << 24);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[j] = o[j];
      }
    }
  }
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
  const int es = elem_bytes(t);
  const bool rows_aligned = aligned16(x) && (ldx * es) % 16 == 0 && (K * es) % 16 == 0;
  if (rows_aligned && perm == nullptr) {
    const int64_t vpr = K * es / 16;
    dim3 grid((unsigned)((vpr + kThreads - 1) / kThreads), (unsigned)(M < 4096 ? M : 4096), 1);
    const uint8_t* xb = static_cast<const uint8_t*>(x);
    if (t == SP24_F16) kept_magnitude_vec_kernel<0><<<grid, kThreads, 0, s>>>(xb, ldx * es, M, vpr, result);
    else if (t == SP24_BF16) kept_magnitude_vec_kernel<1><<<grid, kThreads, 0, s>>>(xb, ldx * es, M, vpr, result);
    else kept_magnitude_vec_kernel<2><<<grid, kThreads, 0, s>>>(xb, ldx * es, M, vpr, result);
    return cuda_status(cudaGetLastError());
  }
  if (rows_aligned && aligned16(perm) && K * es <= 48 * 1024) {
    const unsigned grid = (unsigned)(M < 148 * 8 ? M : 148 * 8);
    const size_t smem = (size_t)K * es;
    const uint8_t* xb = static_cast<const uint8_t*>(x);
    if (t == SP24_F16)
      kept_magnitude_perm_kernel<0, uint16_t><<<grid, kThreads, smem, s>>>(xb, ldx * es, M, K, perm, result);
    else if (t == SP24_BF16)
      kept_magnitude_perm_kernel<1, uint16_t><<<grid, kThreads, smem, s>>>(xb, ldx * es, M, K, perm, result);
    else
      kept_magnitude_perm_kernel<2, int8_t><<<grid, kThreads, smem, s>>>(xb, ldx * es, M, K, perm, result);
    return cuda_status(cudaGetLastError());
  }
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
  const int es = elem_bytes(t);
  if (K % 16 == 0 && aligned16(w) && aligned16(y) && aligned16(meta) && (ldw * es) % 16 == 0 && (ldy * es) % 16 == 0) {
    dim3 grid((unsigned)((K / 16 + kThreads - 1) / kThreads), (unsigned)(M < 8192 ? M : 8192), 1);
    if (es == 2)
      apply_mask_vec_kernel<2><<<grid, kThreads, 0, s>>>((const uint8_t*)w, ldw * es, (const uint8_t*)meta, (int)l,
                                                         (uint8_t*)y, ldy * es, M, K, KB);
    else
      apply_mask_vec_kernel<1><<<grid, kThreads, 0, s>>>((const uint8_t*)w, ldw * es, (const uint8_t*)meta, (int)l,
                                                         (uint8_t*)y, ldy * es, M, K, KB);
    return cuda_status(cudaGetLastError());
  }
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
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t br = M / 4, bc = K / 4;
  const dim3 blocks((unsigned)((bc + kThreads - 1) / kThreads), (unsigned)(br < 16384 ? br : 16384), 1);
  if (t == SP24_F16)
    prune_2d_kernel<0, uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, (uint16_t*)y, ldy, br, bc);
  else if (t == SP24_BF16)
    prune_2d_kernel<1, uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, (uint16_t*)y, ldy, br, bc);
  else
    prune_2d_kernel<2, int8_t><<<blocks, kThreads, 0, s>>>((const int8_t*)x, ldx, (int8_t*)y, ldy, br, bc);
  return cuda_status(cudaGetLastError());
}
