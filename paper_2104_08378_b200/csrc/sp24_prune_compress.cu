// Streaming kernels of the 2:4 path: magnitude pruning (Section 4.1 step 2), compression to
// kept values + 2-bit position metadata and its inverse (Section 3.1, Figure 1), and the
// im2col lowering of a 3x3 convolution (Section 4.2).  All of them are bound by HBM bandwidth:
// every thread moves whole 16-byte vectors, the selection is a handful of integer compares.
#include "sp24_common.cuh"

namespace sp24 {
namespace {

constexpr int kThreads = 256;

// ---- selection -------------------------------------------------------------------------
// Bit p of the result is set iff position p of the group is kept.  Position a beats position b
// (a < b) when key[a] >= key[b] -- equal magnitudes go to the lower index -- so the six
// comparisons define a strict total order and exactly two positions are beaten fewer than
// two times.
__device__ __forceinline__ uint32_t keep_mask4(uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3) {
  uint32_t c01 = k0 >= k1, c02 = k0 >= k2, c03 = k0 >= k3;
  uint32_t c12 = k1 >= k2, c13 = k1 >= k3, c23 = k2 >= k3;
  uint32_t b0 = 3u - (c01 + c02 + c03);
  uint32_t b1 = c01 + 2u - (c12 + c13);
  uint32_t b2 = c02 + c12 + 1u - c23;
  uint32_t b3 = c03 + c13 + c23;
  return (b0 < 2u) | ((b1 < 2u) << 1) | ((b2 < 2u) << 2) | ((b3 < 2u) << 3);
}

// keep mask (two bits set) -> metadata nibble p0 | p1 << 2.
__device__ __forceinline__ uint32_t mask_to_nibble(uint32_t mask) {
  uint32_t p0 = __ffs(mask) - 1, p1 = 31 - __clz(mask);
  return p0 | (p1 << 2);
}

// Which of a group's four 16-bit values (two words: lo = elements 0,1; hi = elements 2,3) are non-zero.
struct Group16 {
  static __device__ __forceinline__ uint32_t nonzero(uint32_t lo, uint32_t hi) {
    return ((lo & 0x7FFFu) != 0) | (((lo >> 16) & 0x7FFFu) != 0) << 1 | ((hi & 0x7FFFu) != 0) << 2 |
           (((hi >> 16) & 0x7FFFu) != 0) << 3;
  }
};

// Which of a group's four int8 values (one word) are non-zero.
struct Group8 {
  static __device__ __forceinline__ uint32_t nonzero(uint32_t w) {
    return ((w & 0xFFu) != 0) | ((w & 0xFF00u) != 0) << 1 | ((w & 0xFF0000u) != 0) << 2 |
           ((w & 0xFF000000u) != 0) << 3;
  }
};

// Magnitude keys of 8-bit elements: |x| for int8 (-128 -> 0x80 = 128, no saturation), the seven
// bits below the sign for the 8-bit floating-point types (`f8` != 0).
__device__ __forceinline__ uint32_t keys8(uint32_t w, int f8) { return f8 ? (w & 0x7F7F7F7Fu) : __vabs4(w); }
__device__ __forceinline__ uint32_t key8(uint32_t e, int f8) { return f8 ? (e & 0x7Fu) : (uint32_t)abs((int)(int8_t)e); }

__device__ __forceinline__ uint4 ld_stream(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void st_stream(void* p, uint4 v) { __stcs(reinterpret_cast<uint4*>(p), v); }

// ---- prune -----------------------------------------------------------------------------
// Any alignment / leading dimension: one thread per group, element-wise accesses.
template <typename T>
__global__ void prune_scalar_kernel(const T* __restrict__ x, int64_t ldx, T* y, int64_t ldy, int64_t groups_per_row,
                                    int64_t total, int f8) {
  int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= total) return;
  int64_t row = id / groups_per_row, g = id - row * groups_per_row;
  const T* src = x + row * ldx + 4 * g;
  T e[4];
  uint32_t key[4];
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    e[p] = src[p];
    key[p] = sizeof(T) == 2 ? (uint32_t)((uint16_t)e[p] & 0x7FFFu) : key8((uint32_t)(uint8_t)e[p], f8);
  }
  uint32_t m = keep_mask4(key[0], key[1], key[2], key[3]);
  T* dst = y + row * ldy + 4 * g;
#pragma unroll
  for (int p = 0; p < 4; ++p) dst[p] = (m >> p) & 1u ? e[p] : (T)0;
}

// ---- metadata addressing ------------------------------------------------------------------
// Byte offset of the 16 metadata bits of chunk `chunk` (16 consecutive columns of A = four
// groups) of row `row`.  Canonical: K/8 bytes per row.  Operand order: 2048-byte blocks of 128
// rows x 128 columns, block (mb, kb) at (mb * KB + kb) * 2048.  Inside a block a 16-bit-type row
// r shares 32-bit words with row r+8 of its 16-row band, the second 16-column half of every
// 32-column slice lives 128 bytes further on, and each 32-column slice is one 32-bit tensor-
// memory column; an int8 row is simply 16 consecutive bytes.
template <int ES>
__device__ __forceinline__ int64_t meta_offset(int layout, int64_t row, int64_t chunk, int64_t K, int64_t KB) {
  if (layout == SP24_META_CANONICAL) return row * (K >> 3) + 2 * chunk;
  int64_t blk = (row >> 7) * KB + (chunk >> 3);
  int r = (int)(row & 127), cl = (int)(chunk & 7);
  int in_blk = ES == 2 ? 16 * (r & 7) + 2 * ((r >> 3) & 1) + 256 * (r >> 4) + 128 * (cl & 1) + 4 * (cl >> 1)
                       : 16 * r + 2 * cl;
  return blk * 2048 + in_blk;
}

// ---- compress (fused prune + compress) ----------------------------------------------------
// The domain is padded (rows to rows_pad, 16-column chunks to chunks_pad) so that the operand-
// order layout gets its 0x4 padding nibbles from the same launch.  Every thread issues all of
// its loads before it consumes any of them.
//
// Selection by table: the six comparisons of a group are made two at a time on packed 15-bit
// keys -- ((a | 0x8000) - b) has bit 15 set iff a >= b, and two such differences fit one 32-bit
// subtraction without a borrow between the halves -- and their six result bits index a 64-entry
// table in shared memory that holds, per outcome, the metadata nibble, the keep mask and the
// byte-permute selectors that gather the two kept values.
__device__ __forceinline__ uint32_t selection_entry(uint32_t idx) {
  // idx bits: 0 = c01, 1 = c03, 2 = c02, 3 = c23, 4 = c12, 5 = c13   (cab: key[a] >= key[b])
  uint32_t c01 = idx & 1, c03 = (idx >> 1) & 1, c02 = (idx >> 2) & 1;
  uint32_t c23 = (idx >> 3) & 1, c12 = (idx >> 4) & 1, c13 = (idx >> 5) & 1;
  uint32_t b0 = 3u - (c01 + c02 + c03), b1 = c01 + 2u - (c12 + c13);
  uint32_t b2 = c02 + c12 + 1u - c23, b3 = c03 + c13 + c23;
  uint32_t mask = (b0 < 2u) | ((b1 < 2u) << 1) | ((b2 < 2u) << 2) | ((b3 < 2u) << 3);
  if (__popc(mask) != 2) mask = 3;  // comparison outcomes no real keys can produce
  uint32_t p0 = __ffs(mask) - 1, p1 = 31 - __clz(mask);
  uint32_t sel8 = p0 | (p1 << 4);                                                // bytes p0, p1 of a word
  uint32_t sel16 = (2 * p0) | ((2 * p0 + 1) << 4) | ((2 * p1) << 8) | ((2 * p1 + 1) << 12);  // halves p0, p1 of a pair
  return (p0 | (p1 << 2)) | (mask << 4) | (sel8 << 8) | (sel16 << 16);
}

__device__ __forceinline__ void build_selection_table(uint32_t* table) {
  int t = threadIdx.y * blockDim.x + threadIdx.x;
  if (t < 64) table[t] = selection_entry((uint32_t)t);
  __syncthreads();
}

// k_lo = [key0, key1], k_hi = [key2, key3] as 16-bit lanes, every key < 2^15.
__device__ __forceinline__ uint32_t selection_index(uint32_t k_lo, uint32_t k_hi) {
  const uint32_t g = 0x80008000u;
  uint32_t r1 = (k_lo | g) - k_hi;                              // bit 15: c02, bit 31: c13
  uint32_t r2 = (k_lo | g) - __byte_perm(k_hi, 0, 0x1032);      // bit 15: c03, bit 31: c12
  uint32_t r3 = (__byte_perm(k_lo, k_hi, 0x5410) | g) - __byte_perm(k_lo, k_hi, 0x7632);  // bit 15: c01, 31: c23
  uint32_t t = (r1 & g) | ((r2 & g) >> 1) | ((r3 & g) >> 2);    // bits 15..13: c02 c03 c01, 31..29: c13 c12 c23
  return ((t >> 13) & 7u) | ((t >> 26) & 0x38u);
}

// 16-bit types: the table indices of the two groups of one 16-byte vector at once.  lo/hi are the masked
// key words of group 0 (k0k1, k2k3) and group 1; word p of the transposed form holds key p of both groups,
// so each of the six comparisons is one subtraction for the two groups.
__device__ __forceinline__ void selection_index_x2(uint32_t lo0, uint32_t hi0, uint32_t lo1, uint32_t hi1,
                                                   uint32_t& idx0, uint32_t& idx1) {
  const uint32_t p0 = __byte_perm(lo0, lo1, 0x5410), p1 = __byte_perm(lo0, lo1, 0x7632);
  const uint32_t p2 = __byte_perm(hi0, hi1, 0x5410), p3 = __byte_perm(hi0, hi1, 0x7632);
  const uint32_t g = 0x80008000u;
  const uint32_t c01 = ((p0 | g) - p1) & g, c02 = ((p0 | g) - p2) & g, c03 = ((p0 | g) - p3) & g;
  const uint32_t c12 = ((p1 | g) - p2) & g, c13 = ((p1 | g) - p3) & g, c23 = ((p2 | g) - p3) & g;
  const uint32_t x = (c01 >> 15) | (c03 >> 14) | (c02 >> 13) | (c23 >> 12) | (c12 >> 11) | (c13 >> 10);
  idx0 = x & 0xFFFFu;
  idx1 = x >> 16;
}

// 8-bit types: the table indices of the four groups of one 16-byte vector at once.  a[g] holds the four
// keys of group g, one per byte.  With all keys below 128 the keys are transposed (word p = key p of
// the four groups) and each of the six comparisons is one byte-wise subtraction with a guard bit,
// ((x | 0x80) - y) bit 7 = (x >= y); the six flag words are merged into one index byte per group.  A
// key of 128 (int8 -128) does not fit the guard trick: such a vector takes the group-by-group path.
__device__ __forceinline__ void selection_index_x4(const uint32_t (&a)[4], uint32_t (&idx)[4]) {
  if ((a[0] | a[1] | a[2] | a[3]) & 0x80808080u) {
#pragma unroll
    for (int g = 0; g < 4; ++g) idx[g] = selection_index(__byte_perm(a[g], 0, 0x4140), __byte_perm(a[g], 0, 0x4342));
    return;
  }
  const uint32_t t0 = __byte_perm(a[0], a[1], 0x5140), t1 = __byte_perm(a[2], a[3], 0x5140);
  const uint32_t t2 = __byte_perm(a[0], a[1], 0x7362), t3 = __byte_perm(a[2], a[3], 0x7362);
  const uint32_t p0 = __byte_perm(t0, t1, 0x5410), p1 = __byte_perm(t0, t1, 0x7632);
  const uint32_t p2 = __byte_perm(t2, t3, 0x5410), p3 = __byte_perm(t2, t3, 0x7632);
  const uint32_t g = 0x80808080u;
  const uint32_t c01 = ((p0 | g) - p1) & g, c02 = ((p0 | g) - p2) & g, c03 = ((p0 | g) - p3) & g;
  const uint32_t c12 = ((p1 | g) - p2) & g, c13 = ((p1 | g) - p3) & g, c23 = ((p2 | g) - p3) & g;
  // index bits: 0 = c01, 1 = c03, 2 = c02, 3 = c23, 4 = c12, 5 = c13 (see selection_entry); byte g of x = group g
  const uint32_t x = (c01 >> 7) | (c03 >> 6) | (c02 >> 5) | (c23 >> 4) | (c12 >> 3) | (c13 >> 2);
  idx[0] = x & 0xFFu;
  idx[1] = (x >> 8) & 0xFFu;
  idx[2] = (x >> 16) & 0xFFu;
  idx[3] = x >> 24;
}

// ---- prune (vectorised) -------------------------------------------------------------------------
// Launch geometry of the vectorised kernels: blockDim = (TX, 256/TX), a warp always lies inside
// one row; thread (tx, ty) of block (bx, by) handles units (bx*UNROLL + u)*TX + tx, u < UNROLL, of
// rows by*TY + ty, + gridDim.y*TY, ...  No integer division on the device.
//
// Per comparison outcome the byte-permute selectors that copy the kept elements and zero the others
// (selector nibble 4 = a zero byte of the second operand): 16-bit types need one selector for each
// of the group's two words, int8 one for its single word.
template <int ES>
__device__ __forceinline__ uint32_t prune_selectors(uint32_t idx) {
  const uint32_t mask = (selection_entry(idx) >> 4) & 0xFu;
  if (ES == 2) {
    uint32_t lo = ((mask & 1u) ? 0x10u : 0x44u) | (((mask & 2u) ? 0x32u : 0x44u) << 8);
    uint32_t hi = ((mask & 4u) ? 0x10u : 0x44u) | (((mask & 8u) ? 0x32u : 0x44u) << 8);
    return lo | (hi << 16);
  }
  return ((mask & 1u) ? 0x0u : 0x4u) | (((mask & 2u) ? 0x1u : 0x4u) << 4) | (((mask & 4u) ? 0x2u : 0x4u) << 8) |
         (((mask & 8u) ? 0x3u : 0x4u) << 12);
}

template <int ES>
__device__ __forceinline__ uint4 prune_vec(uint4 v, const uint32_t* table, int f8) {
  if (ES == 2) {
    uint32_t i0, i1;
    selection_index_x2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu, v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu, i0, i1);
    const uint32_t s0 = table[i0], s1 = table[i1];
    return make_uint4(__byte_perm(v.x, 0, s0 & 0xFFFFu), __byte_perm(v.y, 0, s0 >> 16), __byte_perm(v.z, 0, s1 & 0xFFFFu),
                      __byte_perm(v.w, 0, s1 >> 16));
  }
  uint32_t w[4] = {v.x, v.y, v.z, v.w};
  const uint32_t a[4] = {keys8(w[0], f8), keys8(w[1], f8), keys8(w[2], f8), keys8(w[3], f8)};
  uint32_t idx[4];
  selection_index_x4(a, idx);
#pragma unroll
  for (int g = 0; g < 4; ++g) w[g] = __byte_perm(w[g], 0, table[idx[g]]);
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// One 16-byte vector per thread and unroll step; `vpr` vectors per row.
template <int ES, int UNROLL>
__global__ void __launch_bounds__(kThreads) prune_vec_kernel(const uint8_t* __restrict__ x, int64_t row_bytes_x,
                                                             uint8_t* y, int64_t row_bytes_y, int64_t vpr,
                                                             int64_t rows, int f8) {
  __shared__ uint32_t table[64];
  {
    const int t = threadIdx.y * blockDim.x + threadIdx.x;
    if (t < 64) table[t] = prune_selectors<ES>((uint32_t)t);
    __syncthreads();
  }
  const uint32_t c0 = blockIdx.x * UNROLL * blockDim.x + threadIdx.x;
  for (int64_t row = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; row < rows;
       row += (int64_t)gridDim.y * blockDim.y) {
    const uint8_t* xr = x + row * row_bytes_x;
    uint8_t* yr = y + row * row_bytes_y;
    uint4 v[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const uint32_t c = c0 + u * blockDim.x;
      if (c < vpr) v[u] = ld_stream(xr + c * 16u);
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const uint32_t c = c0 + u * blockDim.x;
      if (c < vpr) st_stream(yr + c * 16u, prune_vec<ES>(v[u], table, f8));
    }
  }
}

template <bool COUNT>
__device__ __forceinline__ void count_dropped(uint32_t lost, unsigned long long* dropped) {
  if (!COUNT) return;
  lost = __reduce_add_sync(0xFFFFFFFFu, lost);
  __shared__ uint32_t warp_sum[kThreads / 32];
  int t = threadIdx.y * blockDim.x + threadIdx.x;
  if ((t & 31) == 0) warp_sum[t >> 5] = lost;
  __syncthreads();
  if (t == 0) {
    uint32_t s = 0;
#pragma unroll
    for (int wi = 0; wi < kThreads / 32; ++wi) s += warp_sum[wi];
    if (s) atomicAdd(dropped, (unsigned long long)s);
  }
}

// 16-bit types.  Work unit: 8 columns (two groups) = one 16-byte load, 8 bytes of values and one
// metadata byte out, so a warp reads 512 and writes 256 contiguous bytes per step.  Lanes 2j and
// 2j+1 hold the two halves of a 16-column chunk; the even lane stores the chunk's 16 metadata bits.
// HW: metadata goes straight into the tensor-core operand order.  FULL: the launch covers exactly
// the matrix (no padding rows / columns, no ragged block), so no bounds are checked.
// PRUNE: the pruned matrix is written as well (y, same shape as x; may be x itself), so that one
// pass over x yields everything the separate prune and compress passes would.
template <int UNROLL, bool COUNT, bool HW, bool FULL, bool PRUNE>
__global__ void __launch_bounds__(kThreads, 4) compress16_kernel(const uint8_t* x, int64_t row_bytes_x,
                                                              uint8_t* __restrict__ vals, int64_t row_bytes_v,
                                                              uint8_t* __restrict__ meta, int64_t M, int64_t K,
                                                              int64_t rows_pad, int64_t chunks_pad,
                                                              unsigned long long* dropped, uint8_t* y,
                                                              int64_t row_bytes_y) {
  __shared__ uint32_t table[64];
  __shared__ uint32_t ptable[PRUNE ? 64 : 1];
  if (PRUNE) {
    const int t = threadIdx.y * blockDim.x + threadIdx.x;
    if (t < 64) ptable[t] = prune_selectors<2>((uint32_t)t);
  }
  build_selection_table(table);
  const uint32_t halves = (uint32_t)(K >> 3), halves_pad = (uint32_t)chunks_pad * 2, KB = (uint32_t)(chunks_pad >> 3);
  const uint32_t h0 = blockIdx.x * UNROLL * blockDim.x + threadIdx.x;
  // metadata offset of this thread's chunks inside a row: fixed for the whole kernel
  uint32_t moff[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    const uint32_t chunk = (h0 + u * blockDim.x) >> 1;
    moff[u] = HW ? (chunk >> 3) * 2048u + 128u * (chunk & 1u) + 4u * ((chunk >> 1) & 3u) : 2u * chunk;
  }
  uint32_t lost = 0;
  for (int64_t row = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; row < rows_pad;
       row += (int64_t)gridDim.y * blockDim.y) {
    const uint8_t* xr = x + row * row_bytes_x;
    uint8_t* vr = vals + row * row_bytes_v;
    const uint32_t r = (uint32_t)row & 127u;
    uint8_t* mr = HW ? meta + (row >> 7) * ((int64_t)KB * 2048) + (16u * (r & 7u) + 2u * ((r >> 3) & 1u) + 256u * (r >> 4))
                     : meta + row * (K >> 3);
    const bool row_live = FULL || row < M;
    uint4 in[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const uint32_t half = h0 + u * blockDim.x;
      if (row_live && (FULL || half < halves)) in[u] = ld_stream(xr + half * 16u);
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const uint32_t half = h0 + u * blockDim.x;
      uint32_t mbyte = 0x44u;  // padding: positions (0, 1) in both groups
      if (row_live && (FULL || half < halves)) {
        const uint32_t w[4] = {in[u].x, in[u].y, in[u].z, in[u].w};
        uint32_t i0, i1;
        selection_index_x2(w[0] & 0x7FFF7FFFu, w[1] & 0x7FFF7FFFu, w[2] & 0x7FFF7FFFu, w[3] & 0x7FFF7FFFu, i0, i1);
        const uint32_t e0 = table[i0], e1 = table[i1];
        if (PRUNE) {
          const uint32_t s0 = ptable[i0], s1 = ptable[i1];
          st_stream(y + row * row_bytes_y + half * 16u,
                    make_uint4(__byte_perm(w[0], 0, s0 & 0xFFFFu), __byte_perm(w[1], 0, s0 >> 16),
                               __byte_perm(w[2], 0, s1 & 0xFFFFu), __byte_perm(w[3], 0, s1 >> 16)));
        }
        __stcs(reinterpret_cast<uint2*>(vr + half * 8u),
               make_uint2(__byte_perm(w[0], w[1], e0 >> 16), __byte_perm(w[2], w[3], e1 >> 16)));
        mbyte = (e0 & 0xFu) | ((e1 & 0xFu) << 4);
        if (COUNT)
          lost += __popc(Group16::nonzero(w[0], w[1]) & ~(e0 >> 4) & 0xFu) +
                  __popc(Group16::nonzero(w[2], w[3]) & ~(e1 >> 4) & 0xFu);
      }
      const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, mbyte, 1);
      if ((threadIdx.x & 1) == 0 && (FULL || half < halves_pad))
        *reinterpret_cast<uint16_t*>(mr + moff[u]) = (uint16_t)(mbyte | (other << 8));
    }
  }
  count_dropped<COUNT>(lost, dropped);
}

// int8.  Work unit: one chunk of 16 columns (four groups) = one 16-byte load, 8 bytes of values and
// 16 bits of metadata out.
template <int UNROLL, bool COUNT, bool HW, bool FULL, bool PRUNE>
__global__ void __launch_bounds__(kThreads, 4) compress8_kernel(const uint8_t* x, int64_t row_bytes_x,
                                                             uint8_t* __restrict__ vals, int64_t row_bytes_v,
                                                             uint8_t* __restrict__ meta, int64_t M, int64_t K,
                                                             int64_t rows_pad, int64_t chunks_pad,
                                                             unsigned long long* dropped, int f8, uint8_t* y,
                                                             int64_t row_bytes_y) {
  __shared__ uint32_t table[64];
  __shared__ uint32_t ptable[PRUNE ? 64 : 1];
  if (PRUNE) {
    const int t = threadIdx.y * blockDim.x + threadIdx.x;
    if (t < 64) ptable[t] = prune_selectors<1>((uint32_t)t);
  }
  build_selection_table(table);
  const uint32_t chunks = (uint32_t)(K >> 4), cpad = (uint32_t)chunks_pad, KB = (uint32_t)(chunks_pad >> 3);
  const uint32_t c0 = blockIdx.x * UNROLL * blockDim.x + threadIdx.x;
  uint32_t moff[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    const uint32_t chunk = c0 + u * blockDim.x;
    moff[u] = HW ? (chunk >> 3) * 2048u + 2u * (chunk & 7u) : 2u * chunk;
  }
  uint32_t lost = 0;
  for (int64_t row = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; row < rows_pad;
       row += (int64_t)gridDim.y * blockDim.y) {
    const uint8_t* xr = x + row * row_bytes_x;
    uint8_t* vr = vals + row * row_bytes_v;
    uint8_t* mr = HW ? meta + (row >> 7) * ((int64_t)KB * 2048) + 16u * ((uint32_t)row & 127u) : meta + row * (K >> 3);
    const bool row_live = FULL || row < M;
    uint4 in[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const uint32_t chunk = c0 + u * blockDim.x;
      if (row_live && (FULL || chunk < chunks)) in[u] = ld_stream(xr + chunk * 16u);
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const uint32_t chunk = c0 + u * blockDim.x;
      if (!FULL && chunk >= cpad) continue;
      uint32_t mbits = 0x4444u;
      if (row_live && (FULL || chunk < chunks)) {
        const uint32_t w[4] = {in[u].x, in[u].y, in[u].z, in[u].w};
        uint32_t out[2] = {0, 0};
        uint32_t pw[4];
        mbits = 0;
        const uint32_t keys[4] = {keys8(w[0], f8), keys8(w[1], f8), keys8(w[2], f8), keys8(w[3], f8)};
        uint32_t idx4[4];
        selection_index_x4(keys, idx4);
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const uint32_t a = keys[g];
          const uint32_t idx = idx4[g];
          const uint32_t e = table[idx];
          if (PRUNE) pw[g] = __byte_perm(w[g], 0, ptable[idx]);
          const uint32_t pair = __byte_perm(w[g], 0, ((e >> 8) & 0xFFu) | 0x4400u);
          out[g >> 1] |= pair << (16 * (g & 1));
          mbits |= (e & 0xFu) << (4 * g);
          if (COUNT) lost += __popc(Group8::nonzero(a) & ~(e >> 4) & 0xFu);
        }
        __stcs(reinterpret_cast<uint2*>(vr + chunk * 8u), make_uint2(out[0], out[1]));
        if (PRUNE) st_stream(y + row * row_bytes_y + chunk * 16u, make_uint4(pw[0], pw[1], pw[2], pw[3]));
      }
      *reinterpret_cast<uint16_t*>(mr + moff[u]) = (uint16_t)mbits;
    }
  }
  count_dropped<COUNT>(lost, dropped);
}

// Any alignment: one thread per 8 columns (two groups = one metadata byte), element-wise.
template <typename T>
__global__ void compress_scalar_kernel(const T* __restrict__ x, int64_t ldx, T* __restrict__ vals, int64_t ldv,
                                       uint8_t* __restrict__ meta, int layout, int64_t M, int64_t K,
                                       int64_t rows_pad, int64_t bytes_pad, unsigned long long* dropped, int f8) {
  constexpr int ES = sizeof(T);
  const int64_t total = rows_pad * bytes_pad, KB = bytes_pad >> 4;
  int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= total) return;
  int64_t row = id / bytes_pad, bi = id - row * bytes_pad;  // bi: metadata byte index in the row
  uint32_t mbyte = 0x44u, lost = 0;
  if (row < M && bi < (K >> 3)) {
    mbyte = 0;
    for (int h = 0; h < 2; ++h) {
      const T* src = x + row * ldx + 8 * bi + 4 * h;
      T e[4];
      uint32_t key[4];
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        e[p] = src[p];
        key[p] = ES == 2 ? (uint32_t)((uint16_t)e[p] & 0x7FFFu) : key8((uint32_t)(uint8_t)e[p], f8);
      }
      uint32_t m = keep_mask4(key[0], key[1], key[2], key[3]);
      uint32_t nib = mask_to_nibble(m);
      T* dst = vals + row * ldv + 4 * bi + 2 * h;
      dst[0] = e[nib & 3];
      dst[1] = e[nib >> 2];
      mbyte |= nib << (4 * h);
#pragma unroll
      for (int p = 0; p < 4; ++p) lost += (key[p] != 0 && !((m >> p) & 1u));
    }
  }
  int64_t off = meta_offset<ES>(layout, row, bi >> 1, K, KB) + (bi & 1);
  meta[off] = (uint8_t)mbyte;
  if (dropped != nullptr && lost) atomicAdd(dropped, (unsigned long long)lost);
}

// ---- decompress ---------------------------------------------------------------------------
template <int ES>
__global__ void __launch_bounds__(kThreads) decompress_vec_kernel(const uint8_t* __restrict__ vals, int64_t row_bytes_v,
                                                                  const uint8_t* __restrict__ meta, int layout,
                                                                  uint8_t* __restrict__ y, int64_t row_bytes_y,
                                                                  int64_t M, int64_t K, int64_t chunks_pad) {
  // threads along a row (one 16-column chunk each), blockIdx.y strides over the rows: no division
  const int64_t chunks = K >> 4, KB = chunks_pad >> 3;
  const int64_t chunk = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (chunk >= chunks) return;
  for (int64_t row = blockIdx.y; row < M; row += gridDim.y) {
  uint32_t mbits = *reinterpret_cast<const uint16_t*>(meta + meta_offset<ES>(layout, row, chunk, K, KB));
  if (ES == 2) {
    uint4 v = ld_stream(vals + row * row_bytes_v + chunk * 16);
    uint32_t in[4] = {v.x, v.y, v.z, v.w};
    uint32_t w[8];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t nib = (mbits >> (4 * g)) & 0xFu;
      uint64_t both = ((uint64_t)(in[g] & 0xFFFFu) << (16 * (nib & 3))) | ((uint64_t)(in[g] >> 16) << (16 * (nib >> 2)));
      w[2 * g] = (uint32_t)both;
      w[2 * g + 1] = (uint32_t)(both >> 32);
    }
    uint8_t* dst = y + row * row_bytes_y + chunk * 32;
    st_stream(dst, make_uint4(w[0], w[1], w[2], w[3]));
    st_stream(dst + 16, make_uint4(w[4], w[5], w[6], w[7]));
  } else {
    uint2 v = __ldcs(reinterpret_cast<const uint2*>(vals + row * row_bytes_v + chunk * 8));
    uint32_t in[2] = {v.x, v.y};
    uint32_t w[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t nib = (mbits >> (4 * g)) & 0xFu;
      uint32_t pair = (in[g >> 1] >> (16 * (g & 1))) & 0xFFFFu;
      w[g] = ((pair & 0xFFu) << (8 * (nib & 3))) | ((pair >> 8) << (8 * (nib >> 2)));
    }
    st_stream(y + row * row_bytes_y + chunk * 16, make_uint4(w[0], w[1], w[2], w[3]));
  }
  }
}

template <typename T>
__global__ void decompress_scalar_kernel(const T* __restrict__ vals, int64_t ldv, const uint8_t* __restrict__ meta,
                                         int layout, T* __restrict__ y, int64_t ldy, int64_t M, int64_t K,
                                         int64_t bytes_pad) {
  constexpr int ES = sizeof(T);
  const int64_t KB = bytes_pad >> 4, bytes = K >> 3;
  int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= M * bytes) return;
  int64_t row = id / bytes, bi = id - row * bytes;
  uint32_t mbyte = meta[meta_offset<ES>(layout, row, bi >> 1, K, KB) + (bi & 1)];
  for (int h = 0; h < 2; ++h) {
    uint32_t nib = (mbyte >> (4 * h)) & 0xFu;
    const T* src = vals + row * ldv + 4 * bi + 2 * h;
    T* dst = y + row * ldy + 8 * bi + 4 * h;
    T e0 = src[0], e1 = src[1];
#pragma unroll
    for (int p = 0; p < 4; ++p) dst[p] = p == (int)(nib & 3) ? e0 : (p == (int)(nib >> 2) ? e1 : (T)0);
  }
}

// ---- im2col (3x3, stride 1, pad 1, NHWC) ------------------------------------------------------
// Out row = output pixel, out column = (r, s, c).  A block handles the pixels of one image row (n, h):
// blockIdx.x = h, blockIdx.y strides over n, threadIdx = (16-byte vector of channels, filter tap, pixel
// column), so no thread divides anything and a warp writes 512 contiguous bytes.
__global__ void __launch_bounds__(kThreads + 64) im2col_3x3_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out,
                                                                   int64_t row_bytes_out, int64_t Nb, int H, int W,
                                                                   int c_vecs) {
  const int h = blockIdx.x, rs = threadIdx.y, r = rs / 3, s = rs - 3 * r;
  const int hh = h + r - 1;
  const bool row_ok = hh >= 0 && hh < H;
  for (int64_t n = blockIdx.y; n < Nb; n += gridDim.y) {
    const uint8_t* in_row = in + ((n * H + hh) * W) * (int64_t)c_vecs * 16;
    uint8_t* out_row = out + ((n * H + h) * W) * row_bytes_out + (int64_t)rs * c_vecs * 16;
#pragma unroll 4
    for (int w = threadIdx.z; w < W; w += blockDim.z) {
      const int ww = w + s - 1;
      const bool ok = row_ok && ww >= 0 && ww < W;
      for (int cv = threadIdx.x; cv < c_vecs; cv += blockDim.x) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (ok) v = __ldg(reinterpret_cast<const uint4*>(in_row + ((int64_t)ww * c_vecs + cv) * 16));
        st_stream(out_row + w * row_bytes_out + cv * 16, v);
      }
    }
  }
}

// ---- the 1:2 pattern of the TF32 mode (Section 3.2): fp32 storage, one kept value per aligned pair ----
// Metadata: one nibble per pair, 0x4 = first kept, 0xE = second kept (the pair seen as four 16-bit
// halves of which (0,1) or (2,3) survive); canonical K/4 bytes per row, or the operand order of the
// 16-bit types with a nibble standing for a pair (a 2048-byte block = 128 rows x 64 columns).
__device__ __forceinline__ bool keep_second(uint32_t a, uint32_t b) { return (b & 0x7FFFFFFFu) > (a & 0x7FFFFFFFu); }

__global__ void __launch_bounds__(kThreads) prune_f32_kernel(const uint8_t* __restrict__ x, int64_t row_bytes_x, uint8_t* y,
                                                             int64_t row_bytes_y, int64_t vpr, int64_t rows) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= vpr) return;
  for (int64_t row = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; row < rows; row += (int64_t)gridDim.y * blockDim.y) {
    uint4 v = ld_stream(x + row * row_bytes_x + c * 16);
    const bool s0 = keep_second(v.x, v.y), s1 = keep_second(v.z, v.w);
    st_stream(y + row * row_bytes_y + c * 16, make_uint4(s0 ? 0u : v.x, s0 ? v.y : 0u, s1 ? 0u : v.z, s1 ? v.w : 0u));
  }
}

// Work unit: 8 columns (four pairs) = 32 bytes in, 16 bytes of values and 16 bits of metadata out.
template <bool HW>
__global__ void __launch_bounds__(kThreads) compress_f32_kernel(const uint8_t* __restrict__ x, int64_t row_bytes_x,
                                                                uint8_t* __restrict__ vals, int64_t row_bytes_v,
                                                                uint8_t* __restrict__ meta, int64_t M, int64_t K,
                                                                int64_t rows_pad, int64_t chunks_pad,
                                                                unsigned long long* dropped) {
  const uint32_t chunk = blockIdx.x * blockDim.x + threadIdx.x, chunks = (uint32_t)(K >> 3), KB = (uint32_t)(chunks_pad >> 3);
  const uint32_t moff = HW ? (chunk >> 3) * 2048u + 128u * (chunk & 1u) + 4u * ((chunk >> 1) & 3u) : 2u * chunk;
  uint32_t lost = 0;
  for (int64_t row = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; row < rows_pad;
       row += (int64_t)gridDim.y * blockDim.y) {
    if (chunk >= (uint32_t)chunks_pad) continue;
    uint32_t mbits = 0x4444u;
    if (row < M && chunk < chunks) {
      const uint8_t* src = x + row * row_bytes_x + chunk * 32u;
      const uint4 a = ld_stream(src), b = ld_stream(src + 16);
      const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
      uint32_t out[4];
      mbits = 0;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const bool sec = keep_second(w[2 * g], w[2 * g + 1]);
        out[g] = sec ? w[2 * g + 1] : w[2 * g];
        mbits |= (sec ? 0xEu : 0x4u) << (4 * g);
        lost += ((sec ? w[2 * g] : w[2 * g + 1]) & 0x7FFFFFFFu) != 0;
      }
      st_stream(vals + row * row_bytes_v + chunk * 16u, make_uint4(out[0], out[1], out[2], out[3]));
    }
    const uint32_t r = (uint32_t)row & 127u;
    uint8_t* mr = HW ? meta + (row >> 7) * ((int64_t)KB * 2048) + (16u * (r & 7u) + 2u * ((r >> 3) & 1u) + 256u * (r >> 4))
                     : meta + row * (K >> 2);
    *reinterpret_cast<uint16_t*>(mr + moff) = (uint16_t)mbits;
  }
  if (dropped != nullptr && lost) atomicAdd(dropped, (unsigned long long)lost);
}

template <bool HW>
__global__ void __launch_bounds__(kThreads) decompress_f32_kernel(const uint8_t* __restrict__ vals, int64_t row_bytes_v,
                                                                  const uint8_t* __restrict__ meta, uint8_t* __restrict__ y,
                                                                  int64_t row_bytes_y, int64_t M, int64_t K,
                                                                  int64_t chunks_pad) {
  const uint32_t chunk = blockIdx.x * blockDim.x + threadIdx.x, chunks = (uint32_t)(K >> 3), KB = (uint32_t)(chunks_pad >> 3);
  if (chunk >= chunks) return;
  const uint32_t moff = HW ? (chunk >> 3) * 2048u + 128u * (chunk & 1u) + 4u * ((chunk >> 1) & 3u) : 2u * chunk;
  for (int64_t row = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; row < M; row += (int64_t)gridDim.y * blockDim.y) {
    const uint32_t r = (uint32_t)row & 127u;
    const uint8_t* mr = HW ? meta + (row >> 7) * ((int64_t)KB * 2048) + (16u * (r & 7u) + 2u * ((r >> 3) & 1u) + 256u * (r >> 4))
                           : meta + row * (K >> 2);
    const uint32_t mbits = *reinterpret_cast<const uint16_t*>(mr + moff);
    const uint4 v = ld_stream(vals + row * row_bytes_v + chunk * 16u);
    const uint32_t in[4] = {v.x, v.y, v.z, v.w};
    uint32_t w[8];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const bool sec = (((mbits >> (4 * g)) & 3u) >> 1) != 0;
      w[2 * g] = sec ? 0u : in[g];
      w[2 * g + 1] = sec ? in[g] : 0u;
    }
    uint8_t* dst = y + row * row_bytes_y + chunk * 32u;
    st_stream(dst, make_uint4(w[0], w[1], w[2], w[3]));
    st_stream(dst + 16, make_uint4(w[4], w[5], w[6], w[7]));
  }
}

inline unsigned blocks_for(int64_t total, int per_block) { return (unsigned)((total + per_block - 1) / per_block); }

// Block shape and grid of the vectorised kernels for `units` work units per row and `rows` rows:
// TX (a power of two, 32..256) threads along the row, chosen to waste the fewest lanes.
struct RowLaunch {
  dim3 grid, block;
  RowLaunch(int64_t units, int64_t rows, int unroll) {
    int best_tx = 256;
    int64_t best_cover = -1;
    for (int tx = 256; tx >= 32; tx /= 2) {
      int64_t per = (int64_t)tx * unroll;
      int64_t cover = (units + per - 1) / per * per;
      if (best_cover < 0 || cover < best_cover) { best_cover = cover; best_tx = tx; }
    }
    int ty = kThreads / best_tx;
    block = dim3((unsigned)best_tx, (unsigned)ty, 1);
    int64_t gy = (rows + ty - 1) / ty;
    if (gy > 32768) gy = 32768;
    grid = dim3((unsigned)(best_cover / ((int64_t)best_tx * unroll)), (unsigned)gy, 1);
  }
};

}  // namespace

static sp24_status validate_matrix_args(sp24_dtype t, int64_t M, int64_t K, int64_t k_multiple) {
  SP24_RETURN_IF(!is_ab_type(t), SP24_ERR_DTYPE);
  SP24_RETURN_IF(M < 0 || K < 0 || K % k_multiple != 0, SP24_ERR_SHAPE);
  return SP24_OK;
}

}  // namespace sp24

using namespace sp24;

// FP32 storage = the 1:2 pattern of the TF32 mode; vectorised paths only (16-byte aligned, K % 8 == 0).
static sp24_status validate_f32(int64_t M, int64_t K) {
  SP24_RETURN_IF(M < 0 || K < 0 || K % 8 != 0, SP24_ERR_SHAPE);
  return SP24_OK;
}

static dim3 f32_grid(int64_t units, int64_t rows, dim3& block) {
  block = dim3(256, 1, 1);
  if (units <= 128) block = dim3(units <= 32 ? 32 : (units <= 64 ? 64 : 128), 1, 1);
  block.y = kThreads / block.x;
  int64_t gy = (rows + block.y - 1) / block.y;
  if (gy > 32768) gy = 32768;
  return dim3((unsigned)((units + block.x - 1) / block.x), (unsigned)gy, 1);
}

extern "C" sp24_status sp24_prune(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx, void* y,
                                  int64_t ldy, void* stream) {
  if (t == SP24_F32) {
    sp24_status sf = validate_f32(M, K);
    if (sf != SP24_OK) return sf;
    if (M == 0 || K == 0) return SP24_OK;
    SP24_RETURN_IF(x == nullptr || y == nullptr, SP24_ERR_NULL);
    SP24_RETURN_IF(ldx < K || ldy < K || ldx % 4 || ldy % 4, SP24_ERR_STRIDE);
    SP24_RETURN_IF(!aligned16(x) || !aligned16(y), SP24_ERR_ALIGN);
    if ((sf = check_arch()) != SP24_OK) return sf;
    dim3 block, grid = f32_grid(K / 4, M, block);
    prune_f32_kernel<<<grid, block, 0, static_cast<cudaStream_t>(stream)>>>((const uint8_t*)x, ldx * 4, (uint8_t*)y, ldy * 4,
                                                                             K / 4, M);
    return cuda_status(cudaGetLastError());
  }
  sp24_status st = validate_matrix_args(t, M, K, 4);
  if (st != SP24_OK) return st;
  if (M == 0 || K == 0) return SP24_OK;
  SP24_RETURN_IF(x == nullptr || y == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ldx < K || ldy < K, SP24_ERR_STRIDE);
  if ((st = check_arch()) != SP24_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int es = elem_bytes(t), f8 = is_fp8(t) ? 1 : 0;
  const bool vec = aligned16(x) && aligned16(y) && (ldx * es) % 16 == 0 && (ldy * es) % 16 == 0 && (K * es) % 16 == 0;
  if (vec) {
    constexpr int UNROLL = 4;
    int64_t vpr = K * es / 16, rows = M;
    if (ldx == K && ldy == K && vpr < 256 * UNROLL) {  // packed and short rows: fold rows into long ones
      int64_t fold = 1;
      while (vpr * fold * 2 <= 256 * UNROLL && rows % 2 == 0) { fold *= 2; rows /= 2; }
      vpr *= fold;
    }
    RowLaunch L(vpr, rows, UNROLL);
    int64_t rbx = ldx == K && ldy == K ? vpr * 16 : ldx * es, rby = ldx == K && ldy == K ? vpr * 16 : ldy * es;
    if (es == 2)
      prune_vec_kernel<2, UNROLL><<<L.grid, L.block, 0, s>>>((const uint8_t*)x, rbx, (uint8_t*)y, rby, vpr, rows, f8);
    else
      prune_vec_kernel<1, UNROLL><<<L.grid, L.block, 0, s>>>((const uint8_t*)x, rbx, (uint8_t*)y, rby, vpr, rows, f8);
  } else {
    int64_t gpr = K / 4, total = M * gpr;
    unsigned blocks = blocks_for(total, kThreads);
    if (es == 2)
      prune_scalar_kernel<uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, (uint16_t*)y, ldy, gpr, total, 0);
    else
      prune_scalar_kernel<int8_t><<<blocks, kThreads, 0, s>>>((const int8_t*)x, ldx, (int8_t*)y, ldy, gpr, total, f8);
  }
  return cuda_status(cudaGetLastError());
}

namespace sp24 {
namespace {

template <int ES, bool COUNT, bool HW, bool FULL, bool PRUNE>
void launch_compress_vec(const RowLaunch& L, cudaStream_t s, const uint8_t* xs, int64_t rbx, uint8_t* vs, int64_t rbv,
                         uint8_t* ms, int64_t M, int64_t K, int64_t rows_pad, int64_t chunks_pad,
                         unsigned long long* dropped, int f8, uint8_t* ys, int64_t rby) {
  constexpr int UNROLL = 4;
  if (ES == 2)
    compress16_kernel<UNROLL, COUNT, HW, FULL, PRUNE><<<L.grid, L.block, 0, s>>>(xs, rbx, vs, rbv, ms, M, K, rows_pad,
                                                                                chunks_pad, dropped, ys, rby);
  else
    compress8_kernel<UNROLL, COUNT, HW, FULL, PRUNE><<<L.grid, L.block, 0, s>>>(xs, rbx, vs, rbv, ms, M, K, rows_pad,
                                                                               chunks_pad, dropped, f8, ys, rby);
}

// compress (y == nullptr) or fused prune + compress (y = pruned matrix, vector kernels only: returns
// SP24_ERR_UNSUPPORTED when they cannot take the operands) for the 2:4 types.
sp24_status compress_any(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx, void* y, int64_t ldy,
                         void* vals, int64_t ldv, void* meta, sp24_meta_layout l, unsigned long long* dropped,
                         void* stream) {
  sp24_status st = validate_matrix_args(t, M, K, 8);
  if (st != SP24_OK) return st;
  SP24_RETURN_IF(l != SP24_META_CANONICAL && l != SP24_META_TCGEN05, SP24_ERR_UNSUPPORTED);
  if (M == 0 || K == 0) return SP24_OK;
  SP24_RETURN_IF(x == nullptr || vals == nullptr || meta == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ldx < K || ldv < K / 2, SP24_ERR_STRIDE);
  if ((st = check_arch()) != SP24_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int es = elem_bytes(t), f8 = is_fp8(t) ? 1 : 0;
  const bool hw = l == SP24_META_TCGEN05;
  const int64_t rows_pad = hw ? (M + 127) / 128 * 128 : M;
  const int64_t k_pad = hw ? (K + 255) / 256 * 256 : K;
  const bool vec = K % 16 == 0 && aligned16(x) && aligned16(vals) && aligned16(meta) && (ldx * es) % 16 == 0 &&
                   (ldv * es) % (8 * es) == 0;
  if (vec) {
    constexpr int UNROLL = 4;
    const int64_t chunks_pad = k_pad / 16;
    const int64_t units = es == 2 ? chunks_pad * 2 : chunks_pad;  // 16-byte vectors per padded row
    RowLaunch L(units, rows_pad, UNROLL);
    const bool full = rows_pad == M && k_pad == K && units % ((int64_t)L.block.x * UNROLL) == 0;
    const int variant = (y ? 8 : 0) | (dropped ? 4 : 0) | (hw ? 2 : 0) | (full ? 1 : 0);
    const uint8_t* xs = (const uint8_t*)x;
    uint8_t *vs = (uint8_t*)vals, *ms = (uint8_t*)meta, *ys = (uint8_t*)y;
#define SP24_CV(V, COUNT, HW, FULL, PRUNE)                                                                            \
  case V:                                                                                                             \
    if (es == 2)                                                                                                      \
      launch_compress_vec<2, COUNT, HW, FULL, PRUNE>(L, s, xs, ldx * es, vs, ldv * es, ms, M, K, rows_pad, chunks_pad, \
                                                     dropped, f8, ys, ldy * es);                                      \
    else                                                                                                              \
      launch_compress_vec<1, COUNT, HW, FULL, PRUNE>(L, s, xs, ldx * es, vs, ldv * es, ms, M, K, rows_pad, chunks_pad, \
                                                     dropped, f8, ys, ldy * es);                                      \
    break;
    switch (variant) {
      SP24_CV(0, false, false, false, false)
      SP24_CV(1, false, false, true, false)
      SP24_CV(2, false, true, false, false)
      SP24_CV(3, false, true, true, false)
      SP24_CV(4, true, false, false, false)
      SP24_CV(5, true, false, true, false)
      SP24_CV(6, true, true, false, false)
      SP24_CV(7, true, true, true, false)
      SP24_CV(8, false, false, false, true)
      SP24_CV(9, false, false, true, true)
      SP24_CV(10, false, true, false, true)
      SP24_CV(11, false, true, true, true)
      SP24_CV(12, true, false, false, true)
      SP24_CV(13, true, false, true, true)
      SP24_CV(14, true, true, false, true)
      default:
        SP24_CV(15, true, true, true, true)
    }
#undef SP24_CV
  } else {
    if (y != nullptr) return SP24_ERR_UNSUPPORTED;
    int64_t bytes_pad = k_pad / 8, total = rows_pad * bytes_pad;
    unsigned blocks = blocks_for(total, kThreads);
    if (es == 2)
      compress_scalar_kernel<uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)x, ldx, (uint16_t*)vals, ldv,
                                                                   (uint8_t*)meta, (int)l, M, K, rows_pad, bytes_pad,
                                                                   dropped, 0);
    else
      compress_scalar_kernel<int8_t><<<blocks, kThreads, 0, s>>>((const int8_t*)x, ldx, (int8_t*)vals, ldv,
                                                                 (uint8_t*)meta, (int)l, M, K, rows_pad, bytes_pad,
                                                                 dropped, f8);
  }
  return cuda_status(cudaGetLastError());
}

}  // namespace
}  // namespace sp24

extern "C" sp24_status sp24_compress(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx, void* vals,
                                     int64_t ldv, void* meta, sp24_meta_layout l, unsigned long long* dropped,
                                     void* stream) {
  if (t == SP24_F32) {
    sp24_status sf = validate_f32(M, K);
    if (sf != SP24_OK) return sf;
    SP24_RETURN_IF(l != SP24_META_CANONICAL && l != SP24_META_TCGEN05, SP24_ERR_UNSUPPORTED);
    if (M == 0 || K == 0) return SP24_OK;
    SP24_RETURN_IF(x == nullptr || vals == nullptr || meta == nullptr, SP24_ERR_NULL);
    SP24_RETURN_IF(ldx < K || ldv < K / 2 || ldx % 4 || ldv % 4, SP24_ERR_STRIDE);
    SP24_RETURN_IF(!aligned16(x) || !aligned16(vals) || !aligned16(meta), SP24_ERR_ALIGN);
    if ((sf = check_arch()) != SP24_OK) return sf;
    const bool hw = l == SP24_META_TCGEN05;
    const int64_t rows_pad = hw ? (M + 127) / 128 * 128 : M, k_pad = hw ? (K + 127) / 128 * 128 : K;
    dim3 block, grid = f32_grid(k_pad / 8, rows_pad, block);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (hw)
      compress_f32_kernel<true><<<grid, block, 0, s>>>((const uint8_t*)x, ldx * 4, (uint8_t*)vals, ldv * 4, (uint8_t*)meta,
                                                       M, K, rows_pad, k_pad / 8, dropped);
    else
      compress_f32_kernel<false><<<grid, block, 0, s>>>((const uint8_t*)x, ldx * 4, (uint8_t*)vals, ldv * 4, (uint8_t*)meta,
                                                        M, K, rows_pad, k_pad / 8, dropped);
    return cuda_status(cudaGetLastError());
  }
  return compress_any(t, M, K, x, ldx, nullptr, 0, vals, ldv, meta, l, dropped, stream);
}

extern "C" sp24_status sp24_prune_compress(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx, void* y,
                                           int64_t ldy, void* vals, int64_t ldv, void* meta, sp24_meta_layout l,
                                           unsigned long long* dropped, void* stream) {
  const int es = elem_bytes(t);
  const bool fused = is_ab_type(t) && y != nullptr && aligned16(y) && es > 0 && (ldy * es) % 16 == 0 && ldy >= K;
  if (fused) {
    const sp24_status st = compress_any(t, M, K, x, ldx, y, ldy, vals, ldv, meta, l, dropped, stream);
    if (st != SP24_ERR_UNSUPPORTED) return st;
  }
  // no fused kernel for this case (1:2 pattern, or operands the vector kernels cannot take): two passes.
  // compress reads x before prune may overwrite it (y may be x).
  sp24_status st = sp24_compress(t, M, K, x, ldx, vals, ldv, meta, l, dropped, stream);
  if (st != SP24_OK) return st;
  return sp24_prune(t, M, K, x, ldx, y, ldy, stream);
}

extern "C" sp24_status sp24_decompress(sp24_dtype t, int64_t M, int64_t K, const void* vals, int64_t ldv,
                                       const void* meta, sp24_meta_layout l, void* y, int64_t ldy, void* stream) {
  if (t == SP24_F32) {
    sp24_status sf = validate_f32(M, K);
    if (sf != SP24_OK) return sf;
    SP24_RETURN_IF(l != SP24_META_CANONICAL && l != SP24_META_TCGEN05, SP24_ERR_UNSUPPORTED);
    if (M == 0 || K == 0) return SP24_OK;
    SP24_RETURN_IF(y == nullptr || vals == nullptr || meta == nullptr, SP24_ERR_NULL);
    SP24_RETURN_IF(ldy < K || ldv < K / 2 || ldy % 4 || ldv % 4, SP24_ERR_STRIDE);
    SP24_RETURN_IF(!aligned16(y) || !aligned16(vals) || !aligned16(meta), SP24_ERR_ALIGN);
    if ((sf = check_arch()) != SP24_OK) return sf;
    const bool hw = l == SP24_META_TCGEN05;
    const int64_t k_pad = hw ? (K + 127) / 128 * 128 : K;
    dim3 block, grid = f32_grid(K / 8, M, block);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (hw)
      decompress_f32_kernel<true><<<grid, block, 0, s>>>((const uint8_t*)vals, ldv * 4, (const uint8_t*)meta, (uint8_t*)y,
                                                         ldy * 4, M, K, k_pad / 8);
    else
      decompress_f32_kernel<false><<<grid, block, 0, s>>>((const uint8_t*)vals, ldv * 4, (const uint8_t*)meta, (uint8_t*)y,
                                                          ldy * 4, M, K, k_pad / 8);
    return cuda_status(cudaGetLastError());
  }
  sp24_status st = validate_matrix_args(t, M, K, 8);
  if (st != SP24_OK) return st;
  SP24_RETURN_IF(l != SP24_META_CANONICAL && l != SP24_META_TCGEN05, SP24_ERR_UNSUPPORTED);
  if (M == 0 || K == 0) return SP24_OK;
  SP24_RETURN_IF(y == nullptr || vals == nullptr || meta == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ldy < K || ldv < K / 2, SP24_ERR_STRIDE);
  if ((st = check_arch()) != SP24_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int es = elem_bytes(t);
  const bool hw = l == SP24_META_TCGEN05;
  const int64_t k_pad = hw ? (K + 255) / 256 * 256 : K;
  const bool vec = K % 16 == 0 && aligned16(y) && aligned16(vals) && aligned16(meta) && (ldy * es) % 16 == 0 &&
                   (ldv * es) % (8 * es) == 0;
  if (vec) {
    const dim3 blocks((unsigned)((K / 16 + kThreads - 1) / kThreads), (unsigned)(M < 16384 ? M : 16384), 1);
    if (es == 2)
      decompress_vec_kernel<2><<<blocks, kThreads, 0, s>>>((const uint8_t*)vals, ldv * es, (const uint8_t*)meta, (int)l,
                                                           (uint8_t*)y, ldy * es, M, K, k_pad / 16);
    else
      decompress_vec_kernel<1><<<blocks, kThreads, 0, s>>>((const uint8_t*)vals, ldv * es, (const uint8_t*)meta, (int)l,
                                                           (uint8_t*)y, ldy * es, M, K, k_pad / 16);
  } else {
    int64_t total = M * (K / 8);
    unsigned blocks = blocks_for(total, kThreads);
    if (es == 2)
      decompress_scalar_kernel<uint16_t><<<blocks, kThreads, 0, s>>>((const uint16_t*)vals, ldv, (const uint8_t*)meta,
                                                                     (int)l, (uint16_t*)y, ldy, M, K, k_pad / 8);
    else
      decompress_scalar_kernel<int8_t><<<blocks, kThreads, 0, s>>>((const int8_t*)vals, ldv, (const uint8_t*)meta,
                                                                   (int)l, (int8_t*)y, ldy, M, K, k_pad / 8);
  }
  return cuda_status(cudaGetLastError());
}

extern "C" sp24_status sp24_im2col_nhwc_3x3(sp24_dtype t, int64_t Nb, int64_t H, int64_t W, int64_t C, const void* in,
                                            void* out, int64_t ldo, void* stream) {
  SP24_RETURN_IF(!is_ab_type(t), SP24_ERR_DTYPE);
  SP24_RETURN_IF(Nb < 0 || H < 0 || W < 0 || C < 0 || H > (1 << 30) || W > (1 << 30), SP24_ERR_SHAPE);
  const int es = elem_bytes(t);
  SP24_RETURN_IF((C * es) % 16 != 0, SP24_ERR_SHAPE);
  if (Nb == 0 || H == 0 || W == 0 || C == 0) return SP24_OK;
  SP24_RETURN_IF(in == nullptr || out == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ldo < 9 * C || (ldo * es) % 16 != 0, SP24_ERR_STRIDE);
  SP24_RETURN_IF(!aligned16(in) || !aligned16(out), SP24_ERR_ALIGN);
  sp24_status st = check_arch();
  if (st != SP24_OK) return st;
  const int64_t c_vecs = C * es / 16;
  SP24_RETURN_IF(c_vecs > (1 << 24), SP24_ERR_SHAPE);
  const unsigned bx = (unsigned)(c_vecs < 32 ? c_vecs : 32);
  unsigned bz = 288u / (9u * bx);
  bz = bz < 1 ? 1 : (bz > (unsigned)W ? (unsigned)W : bz);
  const dim3 block(bx, 9, bz), grid((unsigned)H, (unsigned)(Nb < 65535 ? Nb : 65535), 1);
  im2col_3x3_kernel<<<grid, block, 0, static_cast<cudaStream_t>(stream)>>>((const uint8_t*)in, (uint8_t*)out, ldo * es, Nb,
                                                                           (int)H, (int)W, (int)c_vecs);
  return cuda_status(cudaGetLastError());
}
