// D = alpha * A * B + beta * C on the sm_100a tensor cores (Section 3.2, Figure 2 of arXiv
// 2104.08378): A is either 2:4-compressed (values + metadata, tcgen05.mma.sp) or dense
// (tcgen05.mma, the "dense variant" that supplies the sparse-vs-dense speedup).
//
// One persistent, warp-specialised kernel:
//   warp 0   TMA producer: compressed-A tiles, metadata blocks and B tiles of one k-block into a
//            ring of shared-memory stages (mbarrier expect_tx / complete_tx);
//   warp 1   MMA issuer (one elected thread): copies the stage's metadata shared -> tensor
//            memory (tcgen05.cp), issues the tcgen05.mma[.sp] of the stage, commits the stage
//            back to the producer and, after the last k-block, the accumulators to the epilogue;
//            owns the tensor-memory allocation;
//   warps 2-9 epilogue, two per tensor-memory lane quarter taking alternate 32-column boxes:
//            tcgen05.ld accumulator -> registers (the next box's load already under way), alpha /
//            beta / conversion in registers, then one of two forms.  Row-major 2-byte outputs: the
//            warps load C and store D themselves, through small per-warp transposing buffers, and
//            hand the accumulators back as soon as their last box is in registers.  Other outputs:
//            a staging box per warp, C boxes TMA-loaded a few boxes ahead, TMA store of the D box.
// CTAS == 2 runs a pair of CTAs (cluster of two): each CTA loads its 128 rows of A / metadata per
// m-block and its half of B, CTA 0 issues cta_group::2 MMAs (M = 256) for both.
// MBLK == 2 gives every CTA two m-blocks (two accumulators, one B tile): what an SM can pull in
// from the L2 per clock, not the tensor pipe, bounds this kernel, and sharing the B tile between
// two m-blocks cuts the bytes per flop by about a third.  The two accumulators then fill tensor
// memory, so the epilogue is not overlapped with the next tile's main loop; MBLK == 1 keeps two
// accumulator buffers and overlaps it.
// Every wait is bounded: on expiry the role records a code in the status record and all roles
// leave through the normal teardown (no trap, no endless spin).  The kernel never clears the
// record: it stays at the first expired wait, across launches, until the host reads it.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "sp24_common.cuh"
#include "sp24_ptx.cuh"

namespace sp24 {
namespace {

constexpr int kBlockM = 128;              // rows of A per CTA and m-block (tensor-memory lanes)
constexpr int kAtomBytes = 128;           // bytes per row of one swizzle-128B operand atom
constexpr int kEpiWarps = 8;              // two per tensor-memory lane quarter, taking alternate boxes
constexpr int kFirstEpiWarp = 2;          // warp 0: TMA producer, warp 1: MMA issuer
constexpr int kNumThreads = 32 * (kFirstEpiWarp + kEpiWarps);
// (Ten warps leave three on two of the SM's four sub-partitions, which caps the kernel at 168
// registers per thread; trading registers between the roles with setmaxnreg was tried and made the
// compiler spill far more than it saved.)
constexpr long long kWaitTimeoutCycles = 2000ll * 1000ll * 1000ll;  // per wait: 1-2 s of SM clock
constexpr uint32_t kTmemCols = 512;

struct GemmParams {
  int64_t M, N, K;
  int64_t ldc, ldd;   // elements
  const void* C;
  void* D;
  uint32_t* status;   // [0] = 0 ok, else code of the first wait that expired; [1] = number of expired waits
  float alpha, beta;
  int32_t m_tiles, n_tiles, k_blocks;
  int32_t meta_kb;    // 128-column metadata blocks per 128-row block (K padded to 256)
  int32_t a_fmt;      // 0 f16, 1 bf16 (kind::f16); ignored for int8
  int32_t cd_type;    // sp24_dtype of C / D
  int32_t has_c;
  int32_t stages, epi_bytes;  // shared memory: ring stages and bytes of epilogue staging
  int32_t epi_lsu;            // epilogue form: 1 = the warps' own loads and stores, 0 = TMA through staging boxes
  long long wait_limit;       // SM cycles after which a device-side wait gives up
  int32_t test_skip_stage;    // test hook: the producers leave out one k-block, so that a wait expires
  int32_t band;       // m-tiles per band of the tile sweep
  int32_t cd_col_major;  // C and D stored M-contiguous (the [tokens, out_features] layout)
  // implicit 3x3 convolution: B is the im2col view of an NHWC activation (never materialised)
  int32_t conv, conv_h, conv_w, conv_c;
  // int8 dequantising epilogue (sp24_gemm_i8_dequant): out = act(row_scale[i] * acc + bias[i]),
  // requantised with out_inv_scale when the output type is int8
  int32_t dequant, relu;
  int32_t acc_f16;    // FP16 accumulation (kind::f16 with a binary16 accumulator; FP16 operands only)
  const float* row_scale;
  const float* bias;
  float out_inv_scale;
};

// MMA kinds: 0 = f16 / bf16, 1 = int8, 2 = tf32, 3 = 8-bit floating point (e4m3 / e5m2)
__host__ __device__ constexpr bool one_byte_operands(int kind) { return kind == 1 || kind == 3; }

template <int KIND, bool SPARSE, int BLOCK_N, int CTAS, int MBLK, bool B_MN>
struct Cfg {
  // 128-byte atoms per stage: sparse A is half as wide as B; the dense variant with two
  // m-blocks takes one atom per operand so that four stages still fit
  static constexpr int kBBoxes = SPARSE ? 2 : (MBLK == 2 ? 1 : 2);
  static constexpr int kABoxes = SPARSE ? 1 : kBBoxes;
  static constexpr int kBRows = BLOCK_N / CTAS;                    // B rows (N) this CTA loads
  static constexpr int kABlockBytes = kABoxes * kBlockM * kAtomBytes;  // one m-block
  static constexpr int kABytes = MBLK * kABlockBytes;
  static constexpr int kAtomElems = KIND == 0 ? 64 : (one_byte_operands(KIND) ? 128 : 32);  // elements per 128-byte row
  static constexpr int kKPerStage = kAtomElems * kBBoxes;  // logical K per stage
  // B with N contiguous (MN-major operand): 128-byte chunks along N, each kKPerStage k-rows of 128 bytes
  static constexpr int kBChunkElems = kAtomElems;
  static constexpr int kBChunks = (kBRows + kBChunkElems - 1) / kBChunkElems;
  static constexpr int kBChunkBytes = kKPerStage * kAtomBytes;
  static constexpr int kBKStepBytes = (SPARSE ? 2 : 1) * (kAtomElems / 4) * kAtomBytes;  // k-rows of one MMA
  // an MN-major tf32 operand exists only in the 128-byte swizzle with 32-byte units (groups of 4 k-rows)
  static constexpr uint32_t kBMnLayout = KIND == 2 ? ptx::kLayoutSw128Base32 : ptx::kLayoutSw128;
  static constexpr uint32_t kBMnSbo = KIND == 2 ? 512 : 1024;
  static constexpr int kBBytes = B_MN ? kBChunks * kBChunkBytes : kBBoxes * kBRows * kAtomBytes;
  static constexpr int kEBlocks = SPARSE ? (one_byte_operands(KIND) ? 2 : 1) : 0;  // 2048-byte metadata blocks per m-block and stage
  static constexpr int kEBlockBytes = kEBlocks * 2048;
  static constexpr int kEBytes = MBLK * kEBlockBytes;
  static constexpr int kEAlloc = (kEBytes + 1023) / 1024 * 1024;
  static constexpr int kStageBytes = kABytes + kBBytes + kEAlloc;
  // shared memory: [stage ring | epilogue staging | barriers]; 1 KB of slack for the 1024-byte alignment
  // The split between ring stages and epilogue staging is made per launch (the output type
  // decides how much staging is useful).
  static constexpr int kSmemLimit = 232448 - 1024 - 512;
  static constexpr int kMaxStages = 8;
  static constexpr int kMinStagesFit = (kSmemLimit - 16384) / kStageBytes;  // with the smallest staging
  static constexpr int kAccStages = MBLK == 2 ? 1 : ((2 * BLOCK_N + (SPARSE ? 32 : 0) <= (int)kTmemCols) ? 2 : 1);
  static constexpr int kECol = kAccStages * MBLK * BLOCK_N;        // first metadata column in tensor memory
  static constexpr int kMmasPerStage = SPARSE ? 4 : 4 * kBBoxes;   // per m-block
  static constexpr int kSmemBytes = 232448;  // always the whole opt-in maximum
  static_assert(kMinStagesFit >= 2, "need at least two stages");
  // the epilogue moves 32-column boxes; a last box of 16 columns (240-column tiles) is handled only by
  // the epilogue for row-major outputs, which bounds every access by the tile's last column
  static_assert(BLOCK_N % 16 == 0, "tile width");
  static_assert(kStageBytes % 1024 == 0, "stages must keep the 1024-byte alignment of the atoms");
  static_assert(kECol + (SPARSE ? 2 * MBLK * 8 : 0) <= (int)kTmemCols, "tensor memory overflow");
};

struct Shared {
  uint64_t full[8], empty[8], tmem_full[2], tmem_empty[2];
  uint64_t c_full[kEpiWarps][4];   // per epilogue warp and staging buffer: C box has landed
  uint32_t tmem_base;
  volatile uint32_t abort;
};
static_assert(sizeof(Shared) <= 512, "barrier block");

__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity, Shared* sh, uint32_t* status,
                                             uint32_t code, long long limit) {
  // fast path: poll a while before any bookkeeping; try_wait itself suspends the thread briefly
#pragma unroll 1
  for (int i = 0; i < 64; ++i)
    if (ptx::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (true) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((++spins & 255u) == 0) {
      if (sh->abort) return false;
      if (clock64() - t0 > limit) {
        sh->abort = 1;
        atomicCAS(status, 0u, code);   // sticky: the first code stays until the host reads and clears it
        atomicAdd(status + 1, 1u);
        return false;
      }
    }
  }
}

// tile index -> (m_tile, n_tile): bands of `band_rows` m-tiles are swept n-tile by n-tile so that
// the tiles in flight at one time share a few A row-panels and B column-panels in the L2; every
// other band is swept from the last n-tile back, so that the first wave of a band uses the B
// columns the last wave of the band before has just read.
__device__ __forceinline__ void tile_coords(int t, int m_tiles, int n_tiles, int band_rows, int& mt, int& nt) {
  int per_band = band_rows * n_tiles;
  int band = t / per_band, in_band = t - band * per_band;
  int rows = min(band_rows, m_tiles - band * band_rows);
  nt = in_band / rows;
  mt = band * band_rows + (in_band - nt * rows);
  if (band & 1) nt = n_tiles - 1 - nt;
}

template <int KIND>
__device__ __forceinline__ uint32_t make_idesc(bool sparse, bool b_mn_major, int a_fmt, int m, int n, bool acc_f16) {
  uint32_t d = 0;
  d |= (sparse ? 1u : 0u) << 2;
  d |= (KIND == 1 ? 2u : (acc_f16 ? 0u : 1u)) << 4;  // accumulator: int32 / fp32 / fp16
  // kind f16: f16 = 0, bf16 = 1; tf32: 2; int8: 1 = signed; 8-bit floats: e4m3 = 0, e5m2 = 1
  uint32_t fmt = (KIND == 0 || KIND == 3) ? (uint32_t)a_fmt : (KIND == 1 ? 1u : 2u);
  d |= fmt << 7;
  d |= fmt << 10;
  d |= (b_mn_major ? 1u : 0u) << 16;               // A is always K-major
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(m >> 4) << 24;
  return d;                                        // no negate, no saturate
}

// ---- epilogue helpers ----------------------------------------------------------------------------
// Dequantising epilogue of the int8 path, all in fp32 and in exactly this order (the int8 output
// is compared bit for bit): t = float(acc) (round to nearest), y = fma(scale, t, bias), optional
// max(y, 0); int8 output: round-to-nearest-even of y * out_inv_scale, clamped to [-127, 127].
__device__ __forceinline__ float dequant_value(uint32_t acc, float scale, float bias, int relu) {
  float y = __fmaf_rn(scale, __int2float_rn((int)acc), bias);
  return relu ? fmaxf(y, 0.f) : y;
}
__device__ __forceinline__ int requant_i8(float y, float inv) {
  int q = __float2int_rn(__fmul_rn(y, inv));
  return max(-127, min(127, q));
}

__device__ __forceinline__ uint32_t pack_16bit(float lo, float hi, bool bf) {
  if (bf) {
    __nv_bfloat162 o = __float22bfloat162_rn(make_float2(lo, hi));
    return *reinterpret_cast<uint32_t*>(&o);
  }
  __half2 o = __float22half2_rn(make_float2(lo, hi));
  return *reinterpret_cast<uint32_t*>(&o);
}
__device__ __forceinline__ float2 unpack_16bit(uint32_t w, bool bf) {
  return bf ? __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w))
            : __half22float2(*reinterpret_cast<const __half2*>(&w));
}

// One thread's row of a 32-column box: out = alpha * acc + beta * c (or the dequantising form) as
// the packed words of the output row: 16 words for 2-byte outputs (CS = 2), 32 for 4-byte ones.
// `c` holds the row's C values in the same packing and is read only if has_c.  One multiply and
// one fused multiply-add per element, whichever path stores the row.
template <int KIND, int CS>
__device__ __forceinline__ void compute_row(const uint32_t (&r)[32], const uint32_t (&c)[8 * CS], bool has_c,
                                            const GemmParams& p, float scale, float bias, uint32_t (&o)[8 * CS]) {
  const bool bf = p.cd_type == SP24_BF16;
  if constexpr (CS == 4) {
    if (KIND == 1 && p.dequant) {
#pragma unroll
      for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(dequant_value(r[e], scale, bias, p.relu));
    } else if (KIND == 1) {
#pragma unroll
      for (int e = 0; e < 32; ++e) o[e] = r[e] + (has_c ? c[e] : 0u);
    } else {
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        float f = __fmul_rn(p.alpha, __uint_as_float(r[e]));
        if (has_c) f = __fmaf_rn(p.beta, __uint_as_float(c[e]), f);
        o[e] = __float_as_uint(f);
      }
    }
  } else {
    if (KIND == 1) {  // dequantised to a 16-bit type (the plain int8 GEMM writes 4-byte results)
#pragma unroll
      for (int e = 0; e < 16; ++e)
        o[e] = pack_16bit(dequant_value(r[2 * e], scale, bias, p.relu), dequant_value(r[2 * e + 1], scale, bias, p.relu), bf);
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        float f0 = __fmul_rn(p.alpha, __uint_as_float(r[2 * e])), f1 = __fmul_rn(p.alpha, __uint_as_float(r[2 * e + 1]));
        if (has_c) {
          const float2 g = unpack_16bit(c[e], bf);
          f0 = __fmaf_rn(p.beta, g.x, f0);
          f1 = __fmaf_rn(p.beta, g.y, f1);
        }
        o[e] = pack_16bit(f0, f1, bf);
      }
    }
  }
}

// FP16 accumulation: every accumulator cell of tensor memory holds a binary16 value in its low half
__device__ __forceinline__ void widen_f16_accumulators(uint32_t (&r)[32]) {
#pragma unroll
  for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__half2float(__ushort_as_half((unsigned short)(r[e] & 0xFFFFu))));
}

// TMA-staged form of a 4-byte row-major box (rows of 128 bytes in the TMA's 128-byte swizzle: 16-byte
// unit v of row r sits at unit v ^ (r & 7), which also keeps the row-per-thread accesses free of bank
// conflicts): C, if any, is in the staging buffer; the result replaces it there.
template <int KIND>
__device__ __forceinline__ void convert_row_staged(const uint32_t (&r)[32], uint8_t* buf, int lane, const GemmParams& p,
                                                   float scale, float bias) {
  uint32_t c[32], o[32];
  uint8_t* row = buf + lane * 128;
  if (p.has_c) {
#pragma unroll
    for (int v = 0; v < 8; ++v) {
      const uint4 x = *reinterpret_cast<const uint4*>(row + ((v ^ (lane & 7)) << 4));
      c[4 * v] = x.x; c[4 * v + 1] = x.y; c[4 * v + 2] = x.z; c[4 * v + 3] = x.w;
    }
  }
  compute_row<KIND, 4>(r, c, p.has_c != 0, p, scale, bias, o);
#pragma unroll
  for (int v = 0; v < 8; ++v)
    *reinterpret_cast<uint4*>(row + ((v ^ (lane & 7)) << 4)) = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
}

// int8 output of the dequantising epilogue: rows of 32 bytes, no swizzle
__device__ __forceinline__ void convert_row_dequant_i8(const uint32_t (&r)[32], uint8_t* buf, int lane, const GemmParams& p,
                                                       float scale, float bias) {
#pragma unroll
  for (int v = 0; v < 2; ++v) {
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      uint32_t word = 0;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        int q = requant_i8(dequant_value(r[16 * v + 4 * e + b], scale, bias, p.relu), p.out_inv_scale);
        word |= ((uint32_t)q & 0xFFu) << (8 * b);
      }
      w[e] = word;
    }
    *reinterpret_cast<uint4*>(buf + lane * 32 + v * 16) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// Column-major output of the dequantising epilogue: box transposed in the staging buffer.
__device__ __forceinline__ void convert_row_dequant_transposed(const uint32_t (&r)[32], uint8_t* buf, int lane,
                                                               const GemmParams& p, float scale, float bias) {
#pragma unroll
  for (int n = 0; n < 32; ++n) {
    const float y = dequant_value(r[n], scale, bias, p.relu);
    if (p.cd_type == SP24_F32) {
      *reinterpret_cast<float*>(buf + n * 128 + ((((lane >> 2) ^ (n & 7))) << 4) + (lane & 3) * 4) = y;
    } else if (p.cd_type == SP24_I8) {
      *reinterpret_cast<int8_t*>(buf + n * 32 + lane) = (int8_t)requant_i8(y, p.out_inv_scale);
    } else {
      uint16_t* u = reinterpret_cast<uint16_t*>(buf + n * 64 + ((((lane >> 3) ^ ((n >> 1) & 3))) << 4) + (lane & 7) * 2);
      if (p.cd_type == SP24_BF16) {
        __nv_bfloat16 o = __float2bfloat16_rn(y);
        *u = *reinterpret_cast<uint16_t*>(&o);
      } else {
        __half o = __float2half_rn(y);
        *u = *reinterpret_cast<uint16_t*>(&o);
      }
    }
  }
}

// Column-major C / D: the staging buffer holds the box transposed (32 rows of n, m contiguous), so
// this thread's 32 values go to 32 different rows, one element each.
template <int KIND>
__device__ __forceinline__ void convert_row_transposed(const uint32_t (&r)[32], uint8_t* buf, int lane,
                                                       const GemmParams& p) {
  const bool wide = KIND == 1 || p.cd_type == SP24_F32;
#pragma unroll
  for (int n = 0; n < 32; ++n) {
    if (wide) {
      uint32_t* u = reinterpret_cast<uint32_t*>(buf + n * 128 + ((((lane >> 2) ^ (n & 7))) << 4) + (lane & 3) * 4);
      if (KIND == 1) {
        *u = r[n] + (p.has_c ? *u : 0u);
      } else {
        float f = p.alpha * __uint_as_float(r[n]);
        if (p.has_c) f += p.beta * __uint_as_float(*u);
        *u = __float_as_uint(f);
      }
    } else {
      uint16_t* u = reinterpret_cast<uint16_t*>(buf + n * 64 + ((((lane >> 3) ^ ((n >> 1) & 3))) << 4) + (lane & 7) * 2);
      float f = p.alpha * __uint_as_float(r[n]);
      if (p.cd_type == SP24_BF16) {
        if (p.has_c) f += p.beta * __bfloat162float(*reinterpret_cast<__nv_bfloat16*>(u));
        __nv_bfloat16 o = __float2bfloat16_rn(f);
        *u = *reinterpret_cast<uint16_t*>(&o);
      } else {
        if (p.has_c) f += p.beta * __half2float(*reinterpret_cast<__half*>(u));
        __half o = __float2half_rn(f);
        *u = *reinterpret_cast<uint16_t*>(&o);
      }
    }
  }
}

// ---- epilogue for row-major C / D of 2- or 4-byte elements ------------------------------------
// The epilogue warps move C and D themselves.  C: every thread loads the 32 values of ITS
// accumulator row straight from global memory into registers, the first boxes of a tile before
// the tile's accumulators are even complete, the later ones a few boxes ahead, so that no load
// latency is left on the path that holds the accumulators (tensor memory cannot be handed back to
// the MMA issuer before it is drained).  D: the row is converted in registers, written to a small
// per-warp buffer in shared memory and read back transposed, so that the global stores of a warp
// cover whole 64-byte row segments.  A "pass" is 32 rows x 64 bytes (2 KB): a whole box of a 2-byte
// type, half a box of a 4-byte type.
template <int KIND, int CS, int BLOCK_N, int CTAS, int MBLK, int ACC_STAGES>
__device__ __forceinline__ void epilogue_rows(const GemmParams& p, Shared* sh, uint8_t* epi, uint32_t tmem_base,
                                              int cta_rank, int cluster_id, int num_clusters, int num_tiles, int warp,
                                              int lane) {
  constexpr int kSub = (BLOCK_N + 31) / 32, kIters = MBLK * kSub;  // the last box of a 240-column tile is half a box
  constexpr int kBoxes = (kIters + 1) / 2;  // boxes per warp and tile (the two warps of a lane quarter alternate)
  constexpr int W = 8 * CS;                 // 32-bit words of one box row
  constexpr int P = CS == 2 ? 4 : 1;        // boxes whose C values are held in registers (16 or 32 registers each)
  constexpr int kPasses = CS / 2;
  constexpr int kUnitElems = 16 / CS;       // elements per 16-byte unit
  const int q = warp & 3, ew = warp - kFirstEpiWarp, half = ew >> 2;
  const int nbuf = p.epi_bytes >= kEpiWarps * 4096 ? 2 : 1;
  uint8_t* stage = epi + ew * (nbuf * 2048);
  const uint8_t* Cb = static_cast<const uint8_t*>(p.C);
  uint8_t* Db = static_cast<uint8_t*>(p.D);
  const size_t ldc_b = (size_t)p.ldc * CS, ldd_b = (size_t)p.ldd * CS;
  const int M = (int)p.M, N = (int)p.N;
  const bool has_c = p.has_c != 0;
  uint32_t creg[P][W];
  int acc = 0;
  uint32_t acc_phase = 0, pass_no = 0;
  for (int t = cluster_id; t < num_tiles && !sh->abort; t += num_clusters) {
    int mt, nt;
    tile_coords(t, p.m_tiles, p.n_tiles, p.band, mt, nt);
    const int col_end = min(N, (nt + 1) * BLOCK_N);  // columns of this tile stop here
    // box n of this warp in this tile: first row / column, accumulator column, inside the matrix?
    auto geom = [&](int n, int& row0, int& col0, int& tcol) -> bool {
      const int it = half + 2 * n;
      const int j = it / kSub, sc = it - j * kSub;
      row0 = ((mt * MBLK + j) * CTAS + cta_rank) * kBlockM + q * 32;
      col0 = nt * BLOCK_N + sc * 32;
      tcol = j * BLOCK_N + sc * 32;
      return it < kIters && row0 < M && col0 < col_end;
    };
    auto load_c = [&](int n, uint32_t (&c)[W]) {
      int row0, col0, tcol;
      if (!geom(n, row0, col0, tcol)) return;
      const int row = row0 + lane;
      if (row >= M) return;
      const uint4* src = reinterpret_cast<const uint4*>(Cb + (size_t)row * ldc_b + (size_t)col0 * CS);
#pragma unroll
      for (int v = 0; v < W / 4; ++v) {
        if (col0 + v * kUnitElems < col_end) {
          const uint4 x = src[v];
          c[4 * v] = x.x; c[4 * v + 1] = x.y; c[4 * v + 2] = x.z; c[4 * v + 3] = x.w;
        }
      }
    };
    if (has_c) {
#pragma unroll
      for (int n = 0; n < P; ++n)
        if (n < kBoxes) load_c(n, creg[n]);
    }
    if (!bounded_wait(&sh->tmem_full[acc], acc_phase, sh, p.status, 4u, p.wait_limit)) break;
    ptx::tc_fence_after();
    const uint32_t t_acc = tmem_base + (acc * MBLK) * BLOCK_N + ((uint32_t)(q * 32) << 16);
    uint32_t racc[2][32];
    {
      int row0, col0, tcol;
      geom(0, row0, col0, tcol);
      ptx::tmem_ld_32x32b_x32(t_acc + tcol, racc[0]);
    }
#pragma unroll
    for (int n = 0; n < kBoxes; ++n) {
      if (half + 2 * n >= kIters) break;  // same answer for the whole warp
      ptx::tmem_ld_wait();
      if (half + 2 * (n + 1) < kIters) {
        int row1, col1, tcol1;
        geom(n + 1, row1, col1, tcol1);
        ptx::tmem_ld_32x32b_x32(t_acc + tcol1, racc[(n + 1) & 1]);
      } else {
        // this warp's part of the accumulators is in registers: hand it back to the MMA issuer (CTA 0 of the pair)
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CTAS == 1) ptx::mbar_arrive(&sh->tmem_empty[acc]);
          else ptx::mbar_arrive_cluster(&sh->tmem_empty[acc], 0);
        }
      }
      int row0, col0, tcol;
      const bool live = geom(n, row0, col0, tcol);  // same answer for the whole warp
      uint32_t o[W];
      if (live) {
        uint32_t (&r)[32] = racc[n & 1];
        if (KIND == 0 && p.acc_f16) widen_f16_accumulators(r);
        float scale = 1.f, bias = 0.f;
        if (KIND == 1 && p.dequant) {
          const int row = min(row0 + lane, M - 1);
          scale = __ldg(p.row_scale + row);
          bias = p.bias ? __ldg(p.bias + row) : 0.f;
        }
        compute_row<KIND, CS>(r, creg[n % P], has_c, p, scale, bias, o);
      }
      // the C registers of box n are free: fetch box n + P into them (also when box n lies outside the matrix)
      if (has_c && n + P < kBoxes) load_c(n + P, creg[n % P]);
      if (live) {
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps) {
          uint8_t* buf = stage + (nbuf == 2 ? (pass_no & 1u) * 2048 : 0);
          if (nbuf == 1) __syncwarp();  // the reads of the previous pass are done
#pragma unroll
          for (int u = 0; u < 4; ++u)
            *reinterpret_cast<uint4*>(buf + lane * 64 + ((u ^ ((lane >> 1) & 3)) << 4)) =
                make_uint4(o[16 * ps + 4 * u], o[16 * ps + 4 * u + 1], o[16 * ps + 4 * u + 2], o[16 * ps + 4 * u + 3]);
          __syncwarp();
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int i = lane + 32 * k, rr = i >> 2, u = i & 3;
            const uint4 x = *reinterpret_cast<const uint4*>(buf + rr * 64 + ((u ^ ((rr >> 1) & 3)) << 4));
            const int grow = row0 + rr, gcol = col0 + ps * (64 / CS) + u * kUnitElems;
            if (grow < M && gcol < col_end) *reinterpret_cast<uint4*>(Db + (size_t)grow * ldd_b + (size_t)gcol * CS) = x;
          }
          ++pass_no;
        }
      }
    }
    if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
  }
}

template <int KIND, bool SPARSE, int BLOCK_N, int CTAS, int MBLK, bool B_MN>
__global__ void __launch_bounds__(kNumThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_e, const __grid_constant__ CUtensorMap map_c,
            const __grid_constant__ CUtensorMap map_d, const GemmParams p) {
  using C = Cfg<KIND, SPARSE, BLOCK_N, CTAS, MBLK, B_MN>;
  extern __shared__ uint8_t smem_raw[];
  // Operand atoms need 1024-byte alignment for the 128-byte swizzle.
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* epi = smem + p.stages * C::kStageBytes;
  Shared* sh = reinterpret_cast<Shared*>(epi + p.epi_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t cta_rank = CTAS == 2 ? ptx::cluster_ctarank() : 0;
  const int cluster_id = blockIdx.x / CTAS, num_clusters = gridDim.x / CTAS;
  const int num_tiles = p.m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(&sh->full[s], 1);
      ptx::mbar_init(&sh->empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&sh->tmem_full[a], 1);
      ptx::mbar_init(&sh->tmem_empty[a], kEpiWarps * CTAS);  // one arrival per epilogue warp of the pair
    }
    for (int w = 0; w < kEpiWarps; ++w)
      for (int b = 0; b < 4; ++b) ptx::mbar_init(&sh->c_full[w][b], 1);
    sh->abort = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&map_a);
    ptx::prefetch_tensormap(&map_b);
    if (SPARSE) ptx::prefetch_tensormap(&map_e);
    if (p.has_c) ptx::prefetch_tensormap(&map_c);
    ptx::prefetch_tensormap(&map_d);
  }
  if (warp == 1) {
    ptx::tmem_alloc<CTAS>(&sh->tmem_base, kTmemCols);
    ptx::tmem_relinquish<CTAS>();
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (CTAS == 2) ptx::cluster_sync();
  ptx::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (ptx::elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      const int box_elems = C::kAtomElems;  // elements per 128-byte atom row
      for (int t = cluster_id; t < num_tiles && !sh->abort; t += num_clusters) {
        int mt, nt;
        tile_coords(t, p.m_tiles, p.n_tiles, p.band, mt, nt);
        // the last n-tile may be narrower: the pair then splits only the columns that exist
        const int n_eff = min(BLOCK_N, (int)(p.N - (int64_t)nt * BLOCK_N));
        const int col0 = nt * BLOCK_N + (int)cta_rank * (n_eff / CTAS);  // first B row (N index)
        // m-blocks of this tile that have rows at all (the rest are neither loaded nor multiplied)
        const int live = min(MBLK, (int)((p.M - (int64_t)mt * MBLK * CTAS * kBlockM + CTAS * kBlockM - 1) /
                                         (CTAS * kBlockM)));
        const uint32_t tx_bytes = (uint32_t)((live * (C::kABlockBytes + C::kEBlockBytes) + C::kBBytes) * CTAS);
        // implicit convolution: (image, row, column) of this CTA's first output pixel
        int conv_n = 0, conv_p = 0, conv_q = 0;
        if (p.conv) {
          conv_n = col0 / (p.conv_h * p.conv_w);
          const int rem = col0 - conv_n * p.conv_h * p.conv_w;
          conv_p = rem / p.conv_w;
          conv_q = rem - conv_p * p.conv_w;
        }
        // (Walking K backwards in every other tile of a CTA, so that a wave first meets the END of the A
        // panel the wave before it has just finished with, saves 12 % of the DRAM reads and 1.5 % of the
        // time, but makes the rounding of a result depend on which CTA computed its tile: the same rows
        // and columns would no longer give the same bits when M or N is split differently.  Not done.)
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!bounded_wait(&sh->empty[stage], phase ^ 1u, sh, p.status, 1u, p.wait_limit)) break;
          if (p.test_skip_stage && t == cluster_id && kb == 1) {
            // test hook: this k-block of the first tile is neither armed nor loaded by either CTA, so
            // the MMA issuer's wait for it expires and every role leaves through the abort path
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
            continue;
          }
          uint8_t* sa = smem + stage * C::kStageBytes;
          uint8_t* sb = sa + C::kABytes;
          uint8_t* se = sb + C::kBBytes;
          uint64_t* full = &sh->full[stage];
          if (cta_rank == 0) ptx::mbar_expect_tx(full, tx_bytes);
#pragma unroll
          for (int j = 0; j < MBLK; ++j) {
            if (j >= live) break;
            const int mb = (mt * MBLK + j) * CTAS + (int)cta_rank;  // 128-row block of A
#pragma unroll
            for (int i = 0; i < C::kABoxes; ++i) {
              uint8_t* dst = sa + j * C::kABlockBytes + i * kBlockM * kAtomBytes;
              int x = (kb * C::kABoxes + i) * box_elems;
              if (CTAS == 1) ptx::tma_load_2d(dst, &map_a, full, x, mb * kBlockM);
              else ptx::tma_load_2d_pair(dst, &map_a, full, 0, x, mb * kBlockM);
            }
            if (SPARSE) {
              // metadata viewed as rows of 128 bytes: block (mb, kb128) starts at row 16 * (mb * KB + kb128)
              int y = 16 * (mb * p.meta_kb + kb * C::kEBlocks);
              if (CTAS == 1) ptx::tma_load_2d(se + j * C::kEBlockBytes, &map_e, full, 0, y);
              else ptx::tma_load_2d_pair(se + j * C::kEBlockBytes, &map_e, full, 0, 0, y);
            }
          }
          if (B_MN) {
            // B stored N-contiguous: boxes of 128 bytes along N x all k-rows of the stage
#pragma unroll
            for (int c = 0; c < C::kBChunks; ++c) {
              int x = col0 + c * C::kBChunkElems, y = kb * C::kKPerStage;
              if (CTAS == 1) ptx::tma_load_2d(sb + c * C::kBChunkBytes, &map_b, full, x, y);
              else ptx::tma_load_2d_pair(sb + c * C::kBChunkBytes, &map_b, full, 0, x, y);
            }
          } else if (p.conv) {
            // k = (r * 3 + s) * C + c: a stage holds channels of one filter tap; rows = output pixels
            const int k0 = kb * C::kKPerStage;
            const int tap = k0 / p.conv_c, c0 = k0 - tap * p.conv_c;
            const int r = tap / 3, sx = tap - 3 * r;
#pragma unroll
            for (int i = 0; i < C::kBBoxes; ++i) {
              uint8_t* dst = sb + i * C::kBRows * kAtomBytes;
              if (CTAS == 1)
                ptx::tma_load_im2col_4d(dst, &map_b, full, c0 + i * box_elems, conv_q - 1, conv_p - 1, conv_n,
                                        (uint16_t)sx, (uint16_t)r);
              else
                ptx::tma_load_im2col_4d_pair(dst, &map_b, full, 0, c0 + i * box_elems, conv_q - 1, conv_p - 1, conv_n,
                                             (uint16_t)sx, (uint16_t)r);
            }
          } else {
#pragma unroll
            for (int i = 0; i < C::kBBoxes; ++i) {
              int x = (kb * C::kBBoxes + i) * box_elems;
              if (CTAS == 1) ptx::tma_load_2d(sb + i * C::kBRows * kAtomBytes, &map_b, full, x, col0);
              else ptx::tma_load_2d_pair(sb + i * C::kBRows * kAtomBytes, &map_b, full, 0, x, col0);
            }
          }
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (cta_rank == 0 && ptx::elect_one()) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0, e_buf = 0;
      for (int t = cluster_id; t < num_tiles && !sh->abort; t += num_clusters) {
        int mt, nt;
        tile_coords(t, p.m_tiles, p.n_tiles, p.band, mt, nt);
        // instruction N = the columns this tile really has (a multiple of 16, of 32 for int8)
        const int n_eff = min(BLOCK_N, (int)(p.N - (int64_t)nt * BLOCK_N));
        const int live = min(MBLK, (int)((p.M - (int64_t)mt * MBLK * CTAS * kBlockM + CTAS * kBlockM - 1) /
                                         (CTAS * kBlockM)));
        const uint32_t idesc = make_idesc<KIND>(SPARSE, B_MN, p.a_fmt, kBlockM * CTAS, n_eff, KIND == 0 && p.acc_f16);
        if (!bounded_wait(&sh->tmem_empty[acc], acc_phase ^ 1u, sh, p.status, 2u, p.wait_limit)) break;
        ptx::tc_fence_after();
        bool ok = true;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!bounded_wait(&sh->full[stage], phase, sh, p.status, 3u, p.wait_limit)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = ptx::smem_u32(smem + stage * C::kStageBytes);
          const uint32_t sb = sa + C::kABytes;
          const uint32_t se = sb + C::kBBytes;
          // metadata columns alternate between two small tensor-memory buffers from k-block to k-block
          const uint32_t e_base = tmem_base + C::kECol + e_buf * (MBLK * 8);
          e_buf ^= 1u;
          if (SPARSE) {
#pragma unroll
            for (int j = 0; j < MBLK; ++j) {
              if (j >= live) break;
#pragma unroll
              for (int i = 0; i < C::kEBlocks; ++i)
                ptx::tmem_cp_128x128b<CTAS>(e_base + j * 8 + 4 * i,
                                            ptx::smem_desc(se + j * C::kEBlockBytes + i * 2048, ptx::kLayoutNone, 128));
            }
          }
#pragma unroll
          for (int j = 0; j < MBLK; ++j) {
            if (j >= live) break;
            const uint32_t d_tmem = tmem_base + (acc * MBLK + j) * BLOCK_N;
            const uint32_t e_tmem = e_base + j * 8;
            const uint32_t saj = sa + j * C::kABlockBytes;
#pragma unroll
            for (int k = 0; k < C::kMmasPerStage; ++k) {
              const uint32_t accumulate = (kb > 0 || k > 0) ? 1u : 0u;
              if (SPARSE) {
                // 32 bytes of compressed A and 64 bytes of B per instruction
                uint64_t da = ptx::smem_desc(saj + k * 32, ptx::kLayoutSw128, 1024);
                uint64_t db = B_MN ? ptx::smem_desc(sb + k * C::kBKStepBytes, C::kBMnLayout, C::kBMnSbo, C::kBChunkBytes)
                                   : ptx::smem_desc(sb + (k >> 1) * C::kBRows * kAtomBytes + (k & 1) * 64, ptx::kLayoutSw128, 1024);
                if (!one_byte_operands(KIND)) {
                  // one 32-bit metadata column per instruction: even-aligned address + selector
                  ptx::mma_sparse<KIND, CTAS>(d_tmem, da, db, e_tmem + (k & ~1), idesc | (uint32_t)(k & 1), accumulate);
                } else {
                  ptx::mma_sparse<KIND, CTAS>(d_tmem, da, db, e_tmem + 2 * k, idesc, accumulate);
                }
              } else {
                uint64_t da = ptx::smem_desc(saj + (k >> 2) * kBlockM * kAtomBytes + (k & 3) * 32, ptx::kLayoutSw128, 1024);
                uint64_t db = B_MN ? ptx::smem_desc(sb + k * C::kBKStepBytes, C::kBMnLayout, C::kBMnSbo, C::kBChunkBytes)
                                   : ptx::smem_desc(sb + (k >> 2) * C::kBRows * kAtomBytes + (k & 3) * 32, ptx::kLayoutSw128, 1024);
                ptx::mma_dense<KIND, CTAS>(d_tmem, da, db, idesc, accumulate);
              }
            }
          }
          // the stage may be refilled once these MMAs have read it
          if (CTAS == 1) ptx::tc_commit(&sh->empty[stage]);
          else ptx::tc_commit_pair(&sh->empty[stage], 3);
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (CTAS == 1) ptx::tc_commit(&sh->tmem_full[acc]);
        else ptx::tc_commit_pair(&sh->tmem_full[acc], 3);
        if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= kFirstEpiWarp) {
    // ------------------------------ epilogue ------------------------------
    const int cs = elem_bytes((sp24_dtype)p.cd_type);
    if (p.epi_lsu) {
      // row-major C / D: loads and stores by the epilogue warps themselves
      if (KIND != 2 && cs == 2)
        epilogue_rows<KIND, 2, BLOCK_N, CTAS, MBLK, C::kAccStages>(p, sh, epi, tmem_base, (int)cta_rank, cluster_id,
                                                                   num_clusters, num_tiles, warp, lane);
      else
        epilogue_rows<KIND, 4, BLOCK_N, CTAS, MBLK, C::kAccStages>(p, sh, epi, tmem_base, (int)cta_rank, cluster_id,
                                                                   num_clusters, num_tiles, warp, lane);
    } else {
    // Column-major C / D, 1-byte outputs, and 4-byte row-major outputs when every epilogue warp can have
    // a box buffer of its own.  Each warp owns 32 accumulator rows and walks its tiles in 32 x 32 boxes:
    // TMA load of the C box (if beta != 0) into a staging buffer a few boxes ahead, tcgen05.ld of the
    // accumulator columns, convert in place, TMA store of the D box.  Boxes outside the matrix are
    // clipped by the TMA.
    const int q = warp & 3;  // tensor-memory lane quarter this warp may read
    const int ew = warp - kFirstEpiWarp;  // epilogue warp 0..7: warps ew and ew + 4 share a lane quarter
    const int buf_bytes = 1024 * cs;
    // Both warps of a quarter work (alternate boxes) when each can have a staging buffer of its own;
    // otherwise the second one only takes part in handing the accumulators back.
    const int split = (p.epi_bytes / kEpiWarps >= buf_bytes) ? 2 : 1;
    const int first_it = ew >> 2;
    const bool active = first_it < split;
    const int warp_bytes = p.epi_bytes / (4 * split);
    const int nbuf = min(4, warp_bytes / buf_bytes);  // staging buffers of this warp: 1, 2 or 4
    const int ahead = nbuf > 1 ? nbuf - 1 : 1;      // boxes the C loads run ahead (their latency is what the epilogue waits on)
    // stores that may still be reading their buffer when the next buffer is claimed: with C the
    // buffer of box seq + ahead is claimed at the end of box seq, without C that of box seq + 1
    const int pending_ok = p.has_c ? nbuf - ahead : nbuf - 1;
    uint8_t* my_bufs = epi + (ew & (4 * split - 1)) * warp_bytes;
    constexpr int kSub = BLOCK_N / 32;
    constexpr int kIters = MBLK * kSub;

    // box `it` of the tile (mt, nt): first row / column and whether any of it lies inside the matrix
    auto box_of = [&](int mt, int nt, int it, int& row0, int& col0) -> bool {
      const int j = it / kSub, sc = it - j * kSub;
      row0 = ((mt * MBLK + j) * CTAS + (int)cta_rank) * kBlockM + q * 32;
      col0 = nt * BLOCK_N + sc * 32;
      return row0 < p.M && col0 < p.N;
    };
    // cursor of the C loads over the same stream of boxes, `ahead` live boxes in front of the consumer
    // (the tile coordinates cost two divisions: once per tile, not per box)
    int pf_t = cluster_id, pf_it = first_it, pf_mt = 0, pf_nt = 0;
    if (pf_t < num_tiles) tile_coords(pf_t, p.m_tiles, p.n_tiles, p.band, pf_mt, pf_nt);
    uint32_t pf_seq = 0;
    auto issue_c_load = [&]() {  // lane 0 only: load the next live box of the stream, if any
      while (pf_t < num_tiles) {
        int row0, col0;
        const bool live_box = box_of(pf_mt, pf_nt, pf_it, row0, col0);
        pf_it += split;
        if (pf_it >= kIters) {
          pf_it = first_it;
          pf_t += num_clusters;
          if (pf_t < num_tiles) tile_coords(pf_t, p.m_tiles, p.n_tiles, p.band, pf_mt, pf_nt);
        }
        if (live_box) {
          const int b = pf_seq % nbuf;
          ptx::mbar_expect_tx(&sh->c_full[ew][b], (uint32_t)buf_bytes);
          ptx::tma_load_2d(my_bufs + b * buf_bytes, &map_c, &sh->c_full[ew][b], p.cd_col_major ? row0 : col0,
                           p.cd_col_major ? col0 : row0);
          ++pf_seq;
          return;
        }
      }
    };
    if (p.has_c && active && lane == 0)
      for (int i = 0; i < ahead; ++i) issue_c_load();

    int acc = 0;
    uint32_t acc_phase = 0, seq = 0;
    for (int t = cluster_id; t < num_tiles && !sh->abort; t += num_clusters) {
      int mt, nt;
      tile_coords(t, p.m_tiles, p.n_tiles, p.band, mt, nt);
      if (!bounded_wait(&sh->tmem_full[acc], acc_phase, sh, p.status, 4u, p.wait_limit)) break;
      ptx::tc_fence_after();
      uint32_t r_next[32];
      const uint32_t t_acc = tmem_base + (acc * MBLK) * BLOCK_N + ((uint32_t)(q * 32) << 16);
      if (active) {
        const int j0 = first_it / kSub, sc0 = first_it - j0 * kSub;
        ptx::tmem_ld_32x32b_x32(t_acc + j0 * BLOCK_N + sc0 * 32, r_next);
      }
      bool ok = true;
#pragma unroll 1
      for (int it = active ? first_it : kIters; it < kIters; it += split) {
        uint32_t r[32];
        ptx::tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 32; ++e) r[e] = r_next[e];
        if (it + split < kIters) {
          const int jn = (it + split) / kSub, scn = (it + split) - jn * kSub;
          ptx::tmem_ld_32x32b_x32(t_acc + jn * BLOCK_N + scn * 32, r_next);
        }
        int row0, col0;
        if (!box_of(mt, nt, it, row0, col0)) continue;  // same answer for the whole warp
        const int b = seq % nbuf;
        uint8_t* buf = my_bufs + b * buf_bytes;
        if (p.has_c && !bounded_wait(&sh->c_full[ew][b], (seq / nbuf) & 1u, sh, p.status, 5u, p.wait_limit)) { ok = false; break; }
        if (KIND == 0 && p.acc_f16) widen_f16_accumulators(r);
        if (KIND == 1 && p.dequant) {
          // this thread's output row: its scale and bias
          const int row = min(row0 + lane, (int)p.M - 1);
          const float scale = __ldg(p.row_scale + row), bias = p.bias ? __ldg(p.bias + row) : 0.f;
          if (p.cd_col_major) convert_row_dequant_transposed(r, buf, lane, p, scale, bias);
          else if (cs == 1) convert_row_dequant_i8(r, buf, lane, p, scale, bias);
          else convert_row_staged<KIND>(r, buf, lane, p, scale, bias);
        } else if (p.cd_col_major) {
          convert_row_transposed<KIND>(r, buf, lane, p);
        } else {
          convert_row_staged<KIND>(r, buf, lane, p, 1.f, 0.f);
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          ptx::tma_store_2d(&map_d, buf, p.cd_col_major ? row0 : col0, p.cd_col_major ? col0 : row0);
          ptx::bulk_commit_group();
          // the buffer claimed next is free once the store that used it last has read it
          if (pending_ok >= 3) ptx::bulk_wait_group_read<3>();
          else if (pending_ok == 2) ptx::bulk_wait_group_read<2>();
          else if (pending_ok == 1) ptx::bulk_wait_group_read<1>();
          else ptx::bulk_wait_group_read<0>();
          if (p.has_c) issue_c_load();
        }
        __syncwarp();
        ++seq;
      }
      if (!ok) break;
      // accumulators drained: hand them back to the MMA issuer (CTA 0 of the pair)
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 1) ptx::mbar_arrive(&sh->tmem_empty[acc]);
        else ptx::mbar_arrive_cluster(&sh->tmem_empty[acc], 0);
      }
      if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) ptx::bulk_wait_group_read<0>();  // staging buffers must outlive the stores that read them
    }
  }

  // ------------------------------ teardown ------------------------------
  ptx::tc_fence_before();
  __syncthreads();
  if (sh->abort) {
    // copies issued before the abort may still be landing in this CTA's shared memory
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  if (CTAS == 2) ptx::cluster_sync();
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc<CTAS>(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

using EncodeIm2colFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

EncodeIm2colFn encode_im2col_fn() {
  static EncodeIm2colFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeIm2colFn>(ptr);
  });
  return fn;
}

// im2col tensor map over an NHWC activation for a 3x3, stride-1, pad-1 convolution: the bounding box
// of the filter's anchor starts one pixel before the image and ends one pixel before its far edge, so
// that anchor + tap (0..2) covers rows/columns -1 .. H, W with zeros outside.
sp24_status make_im2col_map(CUtensorMap* map, const void* x, int es, uint64_t nb, uint64_t h, uint64_t w, uint64_t c,
                            uint32_t channels_per_box, uint32_t pixels_per_box) {
  EncodeIm2colFn fn = encode_im2col_fn();
  if (!fn) return SP24_ERR_CUDA;
  cuuint64_t dims[4] = {c, w, h, nb};
  cuuint64_t strides[3] = {c * es, w * c * es, h * w * c * es};
  int lower[2] = {-1, -1}, upper[2] = {-1, -1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUtensorMapDataType dt = es == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  CUresult r = fn(map, dt, 4, const_cast<void*>(x), dims, strides, lower, upper, channels_per_box, pixels_per_box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SP24_OK : SP24_ERR_CUDA;
}

// 2-D tensor map over a row-major (rows x cols) array of `es`-byte elements with `ld_bytes`
// between rows; box = box_cols x box_rows elements.
constexpr int kSwizzle128Atom32 = 1280;

sp24_status encode_map(CUtensorMap* map, const void* base, int es, uint64_t rows, uint64_t cols, uint64_t ld_bytes,
                       uint32_t box_cols, uint32_t box_rows, int swizzle_bytes) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return SP24_ERR_CUDA;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMapDataType dt = es == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32
                                   : (es == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8);
  // swizzle_bytes: 0, 64, 128, or kSwizzle128Atom32 = the 128-byte pattern in 32-byte units
  CUtensorMapSwizzle sw = swizzle_bytes == kSwizzle128Atom32
                              ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B
                              : (swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                                      : (swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE));
  CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SP24_OK : SP24_ERR_CUDA;
}

// Host-side cache of encoded tensor maps.  A map is a pure function of (address, shape, leading
// dimension, element size, box, swizzle): a layer that is multiplied again with the same buffers
// finds its five maps here instead of encoding them again.  One small table per host thread (no
// lock), replaced round-robin.
struct MapKey {
  const void* base;
  uint64_t rows, cols, ld_bytes;
  uint32_t box_cols, box_rows;
  int32_t es, swizzle;
  bool operator==(const MapKey& o) const {
    return base == o.base && rows == o.rows && cols == o.cols && ld_bytes == o.ld_bytes && box_cols == o.box_cols &&
           box_rows == o.box_rows && es == o.es && swizzle == o.swizzle;
  }
};
struct MapCache {
  static constexpr int kEntries = 32;
  MapKey keys[kEntries];
  CUtensorMap maps[kEntries];
  int used = 0, next = 0;
};

sp24_status make_map(CUtensorMap* map, const void* base, int es, uint64_t rows, uint64_t cols, uint64_t ld_bytes,
                     uint32_t box_cols, uint32_t box_rows, int swizzle_bytes) {
  static thread_local MapCache cache;
  const MapKey key = {base, rows, cols, ld_bytes, box_cols, box_rows, es, swizzle_bytes};
  for (int i = 0; i < cache.used; ++i)
    if (cache.keys[i] == key) {
      *map = cache.maps[i];
      return SP24_OK;
    }
  sp24_status st = encode_map(map, base, es, rows, cols, ld_bytes, box_cols, box_rows, swizzle_bytes);
  if (st != SP24_OK) return st;
  const int slot = cache.used < MapCache::kEntries ? cache.used++ : (cache.next++ % MapCache::kEntries);
  cache.keys[slot] = key;
  cache.maps[slot] = *map;
  return SP24_OK;
}

int sm_count() {
  static std::atomic<int> known[64];
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 1;
  const bool cacheable = dev >= 0 && dev < 64;
  if (cacheable && (n = known[dev].load(std::memory_order_relaxed)) > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 1;
  if (cacheable) known[dev].store(n, std::memory_order_relaxed);
  return n;
}

// Process-wide settings: the benchmarking overrides (environment, read once, or sp24_set_tile_override)
// and the fault-path test hooks (sp24_test_set_fault_hooks only; never read from the environment).
struct Settings {
  std::atomic<int> ctas{0}, block_n{0}, mblk{0}, band{0}, log{0};
  std::atomic<long long> test_wait_cycles{0};
  std::atomic<int> test_skip_stage{0};
};
Settings& settings() {
  static Settings st;
  static std::once_flag once;
  std::call_once(once, [] {
    if (const char* env = getenv("SP24_TILE")) {
      int c = 0, n = 0, m = 1;
      if (sscanf(env, "%dx%dx%d", &c, &n, &m) >= 2) { st.ctas = c; st.block_n = n; st.mblk = m; }
    }
    if (const char* env = getenv("SP24_BAND")) st.band = atoi(env) > 0 ? atoi(env) : 0;
    if (const char* env = getenv("SP24_LOG")) st.log = atoi(env) != 0 || env[0] == '\0' ? 1 : 0;
  });
  return st;
}

template <int KIND, bool SPARSE, int BLOCK_N, int CTAS, int MBLK, bool B_MN>
sp24_status launch(const sp24_gemm_desc* d, const GemmParams& base, const void* A, const void* meta, const void* B,
                   cudaStream_t stream) {
  using C = Cfg<KIND, SPARSE, BLOCK_N, CTAS, MBLK, B_MN>;
  GemmParams p = base;
  const int es = KIND == 0 ? 2 : (one_byte_operands(KIND) ? 1 : 4);
  const int tile_m = kBlockM * CTAS * MBLK;
  p.m_tiles = (int)((d->M + tile_m - 1) / tile_m);
  p.n_tiles = (int)((d->N + BLOCK_N - 1) / BLOCK_N);
  p.k_blocks = (int)((d->K + C::kKPerStage - 1) / C::kKPerStage);
  // metadata blocks per 128-row block: 128 columns each (64 for the 1:2 pattern), an even number of them
  p.meta_kb = KIND == 2 ? (int)(2 * ((d->K + 127) / 128)) : (int)(2 * ((d->K + 255) / 256));
  CUtensorMap map_a, map_b, map_e;
  const uint32_t atom_elems = kAtomBytes / es;
  const uint64_t a_cols = SPARSE ? d->K / 2 : d->K;
  sp24_status st = make_map(&map_a, A, es, d->M, a_cols, d->lda * es, atom_elems, kBlockM, 128);
  if (st != SP24_OK) return st;
  if (p.conv) {
    // B = im2col view of the NHWC activation: boxes of kBRows output pixels x one 128-byte run of channels
    if (B_MN) return SP24_ERR_UNSUPPORTED;
    if (KIND == 2) return SP24_ERR_UNSUPPORTED;
    const uint64_t nb = (uint64_t)d->N / ((uint64_t)p.conv_h * p.conv_w);
    st = make_im2col_map(&map_b, B, es, nb, p.conv_h, p.conv_w, p.conv_c, atom_elems, C::kBRows);
  } else if (B_MN) {
    st = make_map(&map_b, B, es, d->K, d->N, d->ldb * es, C::kBChunkElems, C::kKPerStage,
                  KIND == 2 ? kSwizzle128Atom32 : 128);
  } else {
    st = make_map(&map_b, B, es, d->N, d->K, d->ldb * es, atom_elems, C::kBRows, 128);
  }
  if (st != SP24_OK) return st;
  if (SPARSE) {
    uint64_t meta_rows = (uint64_t)((d->M + 127) / 128) * p.meta_kb * 16;  // rows of 128 bytes
    st = make_map(&map_e, meta, 1, meta_rows, 128, 128, 128, 16 * C::kEBlocks, 0);
    if (st != SP24_OK) return st;
  } else {
    map_e = map_a;
  }
  // C and D move in 32 x 32 boxes whose rows are 64 bytes (2-byte types) or 128 bytes (4-byte types)
  CUtensorMap map_c, map_d;
  const int cs = elem_bytes(d->cd_type);
  const uint64_t cd_rows = p.cd_col_major ? d->N : d->M, cd_cols = p.cd_col_major ? d->M : d->N;
  st = make_map(&map_d, p.D, cs, cd_rows, cd_cols, d->ldd * cs, 32, 32, 32 * cs);
  if (st != SP24_OK) return st;
  if (p.has_c) {
    st = make_map(&map_c, p.C, cs, cd_rows, cd_cols, d->ldc * cs, 32, 32, 32 * cs);
    if (st != SP24_OK) return st;
  } else {
    map_c = map_d;
  }
  // Shared-memory split.  The ring comes first (these kernels are bound by the operand feed: one
  // stage less cost the int8 configuration 9 %); staging gets what is left, up to two boxes per
  // epilogue warp (16 boxes of 1024 output elements), in powers of two from 16 KB.
  {
    p.stages = C::kMinStagesFit > C::kMaxStages ? C::kMaxStages : C::kMinStagesFit;
    const int room = C::kSmemLimit - p.stages * C::kStageBytes;
    // Epilogue form.  Row-major 2-byte outputs: the warps' own loads and stores through two 2 KB
    // transposing buffers per warp (measured against the TMA form: bf16 BERT FFN 26.6 against 28.7 us,
    // fp8 16384 x 8192 x 8192 440 against 472 us, the 256 x 256 x 512 problem 12 against 17 us, the large
    // bf16 GEMM within 3 %).  Row-major 4-byte outputs: TMA boxes if every epilogue warp can have a 4 KB
    // box of its own (int8 4096 x 8192 x 4096: 77 against 80 us), else the warps' own stores (two-m-block
    // int8 tiles, 16 KB of staging: 465 against 504 us on 16384 x 8192 x 8192).  Column-major and 1-byte
    // outputs: TMA boxes, staging in powers of two from 16 KB up to two boxes per epilogue warp.
    int epi = 16384;
    p.epi_lsu = 0;
    if (!p.cd_col_major && cs == 2) {
      p.epi_lsu = 1;
      if (room >= kEpiWarps * 4096) epi = kEpiWarps * 4096;
    } else if (!p.cd_col_major && cs == 4 && room < kEpiWarps * 4096) {
      p.epi_lsu = 1;
    } else {
      while (epi < 16 * 1024 * cs && 2 * epi <= room) epi *= 2;
    }
    p.epi_bytes = epi;
  }
  auto kernel = gemm_kernel<KIND, SPARSE, BLOCK_N, CTAS, MBLK, B_MN>;
  {
    // the shared-memory opt-in is per kernel and device: once is enough
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    SP24_CUDA_CHECK(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(mu);
    if (dev < 0 || dev >= 64 || !done[dev]) {
      SP24_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
      if (dev >= 0 && dev < 64) done[dev] = true;
    }
  }
  const int tiles = p.m_tiles * p.n_tiles;
  int clusters = sm_count() / CTAS;
  if (clusters > tiles) clusters = tiles;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(clusters * CTAS), 1, 1);
  cfg.blockDim = dim3(kNumThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  SP24_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kernel, map_a, map_b, map_e, map_c, map_d, p));
  return SP24_OK;
}

}  // namespace
}  // namespace sp24

using namespace sp24;

extern "C" size_t sp24_gemm_workspace_bytes(const sp24_gemm_desc* d) {
  (void)d;
  return 256;
}

// Tile choice.  Small problems: single CTAs, 128 x 128 tiles.  Otherwise a pair of CTAs, and among the
// pair shapes the one with the smallest estimated time = rounds of tiles over the pairs x time of one
// tile.  The tile times are measured ratios (unit: one 256 x 224 tile per unit of K; interleaved runs on
// 2048..8192-row problems with K = 4096..16384):
//   256 x 224, two accumulator buffers (epilogue overlapped)      K                 the reference
//   256 x 240, the same (16-bit kinds, 16-bit row-major output)    1.04 K            operand bytes per k
//   256 x 256, one accumulator buffer (epilogue exposed)           1.09 K + 450
//   512 x 224, two m-blocks per CTA share a B tile (epilogue exposed): twice the work in
//              1.65 K + 1150 (16-bit kinds), 1.80 K + 820 (8-bit floats), 1.98 K + 200 (int8 -> int32)
// (224: two fp32 accumulators plus the metadata columns fit the 512 columns of tensor memory and 224 is a
// multiple of 32; 240 is the widest multiple of 16 that fits.)  The dense variant: two m-blocks from six
// waves of tiles on, 512 x 256 there (no metadata columns needed); below that the one-m-block width with
// the fewest rounds.
static void choose_tile(const sp24_gemm_desc* d, int& ctas, int& block_n, int& mblk) {
  const int64_t n224 = (d->N + 223) / 224;
  ctas = 1; block_n = 128; mblk = 1;
  if (d->M < 256 || (d->M / 256) * n224 < 32) return;
  ctas = 2; block_n = 224;
  const bool k_major_b = d->order_b == SP24_COL_MAJOR;
  const int64_t pairs = sm_count() / 2 > 0 ? sm_count() / 2 : 1;
  const bool bits16 = d->ab_type == SP24_F16 || d->ab_type == SP24_BF16;
  const bool has_240 = bits16 && k_major_b && d->order_d == SP24_ROW_MAJOR && elem_bytes(d->cd_type) == 2;
  if (d->a_is_dense) {
    if (d->M >= 512 && (d->M / 512) * n224 >= 444) {
      mblk = 2;
      // two 256-column accumulators fill tensor memory exactly: 9 % fewer operand bytes per flop than 512 x 224
      if (k_major_b && d->ab_type != SP24_F32) block_n = 256;
      return;
    }
    // one m-block: the width that needs the fewest rounds of tiles, operand bytes per k as the tie-break
    // (without metadata columns two 256-column accumulators fit, so 256 x 256 keeps its epilogue overlapped)
    const int widths[3] = {224, has_240 ? 240 : 0, k_major_b && d->ab_type != SP24_F32 ? 256 : 0};
    double best = 0.0;
    for (const int bn : widths) {
      if (bn == 0) continue;
      const int64_t tiles = ((d->M + 255) / 256) * ((d->N + bn - 1) / bn);
      const double cost = (double)((tiles + pairs - 1) / pairs) * (256.0 + bn);
      if (best == 0.0 || cost < best) { best = cost; block_n = bn; }
    }
    return;
  }
  const double K = (double)d->K;
  const double two_a = d->ab_type == SP24_I8 ? 1.98 : (is_fp8(d->ab_type) ? 1.80 : 1.65);
  const double two_b = d->ab_type == SP24_I8 ? 200.0 : (is_fp8(d->ab_type) ? 820.0 : 1150.0);
  struct Candidate { int block_n, mblk; bool built; double tile_time; };
  const Candidate candidates[4] = {
      {224, 2, d->M >= 512, two_a * K + two_b},
      {224, 1, true, K},
      {240, 1, has_240, (144.0 + 240.0) / (144.0 + 224.0) * K},
      {256, 1, k_major_b && (bits16 || d->N <= 2048), (144.0 + 256.0) / (144.0 + 224.0) * K + 450.0},
  };
  double best = 0.0;
  for (const Candidate& c : candidates) {
    if (!c.built) continue;
    const int64_t rows = 256 * c.mblk;
    const int64_t tiles = ((d->M + rows - 1) / rows) * ((d->N + c.block_n - 1) / c.block_n);
    const double cost = (double)((tiles + pairs - 1) / pairs) * c.tile_time;
    if (best == 0.0 || cost < best) { best = cost; block_n = c.block_n; mblk = c.mblk; }
  }
}

extern "C" sp24_status sp24_gemm_plan(const sp24_gemm_desc* d, int* ctas, int* block_n, int* mblk) {
  SP24_RETURN_IF(d == nullptr || ctas == nullptr || block_n == nullptr || mblk == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(d->M <= 0 || d->N <= 0 || d->K <= 0, SP24_ERR_SHAPE);
  choose_tile(d, *ctas, *block_n, *mblk);
  Settings& cfg = settings();
  if (const int c = cfg.ctas.load(std::memory_order_relaxed)) {
    *ctas = c;
    *block_n = cfg.block_n.load(std::memory_order_relaxed);
    *mblk = cfg.mblk.load(std::memory_order_relaxed);
  }
  return SP24_OK;
}

static sp24_status validate_gemm(const sp24_gemm_desc* d, const void* alpha, const void* A, const void* meta,
                                 const void* B, const void* beta, const void* C, void* D, void* ws, size_t ws_bytes,
                                 bool& has_c, float& falpha, float& fbeta, bool dequant = false) {
  SP24_RETURN_IF(d == nullptr || (!dequant && (alpha == nullptr || beta == nullptr)), SP24_ERR_NULL);
  const bool tf32 = d->ab_type == SP24_F32;
  const bool f8 = is_fp8(d->ab_type);
  const bool fp = d->ab_type == SP24_F16 || d->ab_type == SP24_BF16 || tf32 || f8;
  SP24_RETURN_IF(!fp && d->ab_type != SP24_I8, SP24_ERR_DTYPE);
  SP24_RETURN_IF(tf32 && d->cd_type != SP24_F32, SP24_ERR_UNSUPPORTED);
  if (dequant)
    SP24_RETURN_IF(fp || (d->cd_type != SP24_BF16 && d->cd_type != SP24_F16 && d->cd_type != SP24_F32 &&
                          d->cd_type != SP24_I8),
                   SP24_ERR_DTYPE);
  else if (f8) SP24_RETURN_IF(d->cd_type != SP24_F16 && d->cd_type != SP24_BF16 && d->cd_type != SP24_F32, SP24_ERR_DTYPE);
  else if (fp) SP24_RETURN_IF(d->cd_type != d->ab_type && d->cd_type != SP24_F32, SP24_ERR_DTYPE);
  else SP24_RETURN_IF(d->cd_type != SP24_I32, SP24_ERR_DTYPE);
  const int64_t mult = elem_bytes(d->ab_type) == 1 ? 32 : 16;
  SP24_RETURN_IF(d->M < 0 || d->N < 0 || d->K <= 0, SP24_ERR_SHAPE);
  SP24_RETURN_IF(d->M % mult || d->N % mult || d->K % mult, SP24_ERR_SHAPE);
  SP24_RETURN_IF(d->M > (int64_t(1) << 30) || d->N > (int64_t(1) << 30) || d->K > (int64_t(1) << 30), SP24_ERR_SHAPE);
  SP24_RETURN_IF(d->order_b != SP24_COL_MAJOR && d->order_b != SP24_ROW_MAJOR, SP24_ERR_UNSUPPORTED);
  SP24_RETURN_IF(d->order_d != SP24_ROW_MAJOR && d->order_d != SP24_COL_MAJOR, SP24_ERR_UNSUPPORTED);
  if (dequant) {
    falpha = 1.f;
    fbeta = 0.f;
  } else if (fp) {
    falpha = *static_cast<const float*>(alpha);
    fbeta = *static_cast<const float*>(beta);
  } else {
    int32_t ia = *static_cast<const int32_t*>(alpha), ib = *static_cast<const int32_t*>(beta);
    SP24_RETURN_IF(ia != 1 || (ib != 0 && ib != 1), SP24_ERR_UNSUPPORTED);
    falpha = 1.f;
    fbeta = (float)ib;
  }
  has_c = fbeta != 0.f;
  // C is converted in place into D inside the epilogue's staging buffer: same order for both
  SP24_RETURN_IF(has_c && d->order_c != d->order_d, SP24_ERR_UNSUPPORTED);
  if (d->M == 0 || d->N == 0) return SP24_OK;
  SP24_RETURN_IF(A == nullptr || B == nullptr || D == nullptr || (has_c && C == nullptr), SP24_ERR_NULL);
  SP24_RETURN_IF(!d->a_is_dense && meta == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(ws == nullptr || ws_bytes < 256 || !aligned16(ws), SP24_ERR_WORKSPACE);
  const int es = elem_bytes(d->ab_type), cs = elem_bytes(d->cd_type);
  const int64_t a_cols = d->a_is_dense ? d->K : d->K / 2;
  const int64_t cd_width = d->order_d == SP24_COL_MAJOR ? d->M : d->N;
  SP24_RETURN_IF(d->lda < a_cols || d->ldb < (d->order_b == SP24_COL_MAJOR ? d->K : d->N) || d->ldd < cd_width ||
                     (has_c && d->ldc < cd_width),
                 SP24_ERR_STRIDE);
  SP24_RETURN_IF((d->lda * es) % 16 || (d->ldb * es) % 16 || (d->ldd * cs) % 16 || (has_c && (d->ldc * cs) % 16),
                 SP24_ERR_STRIDE);
  SP24_RETURN_IF(!aligned16(A) || !aligned16(B) || !aligned16(D) || (has_c && !aligned16(C)) ||
                     (!d->a_is_dense && !aligned16(meta)),
                 SP24_ERR_ALIGN);
  return SP24_OK;
}

struct ConvArgs {
  int64_t nb, h, w, c;
};

struct DequantArgs {
  const float* row_scale;
  const float* bias;
  int relu;
  float out_inv_scale;
};

static sp24_status run_gemm(const sp24_gemm_desc* d, const void* alpha, const void* A, const void* meta, const void* B,
                            const void* beta, const void* C, void* D, void* workspace, size_t workspace_bytes,
                            void* stream, const DequantArgs* dq, const ConvArgs* cv = nullptr, bool acc_f16 = false) {
  bool has_c = false;
  float falpha = 1.f, fbeta = 0.f;
  sp24_status st = validate_gemm(d, alpha, A, meta, B, beta, C, D, workspace, workspace_bytes, has_c, falpha, fbeta,
                                 dq != nullptr);
  if (st != SP24_OK) return st;
  if (d->M == 0 || d->N == 0) return SP24_OK;
  if ((st = check_arch()) != SP24_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  GemmParams p = {};
  if (cv) {
    p.conv = 1;
    p.conv_h = (int)cv->h;
    p.conv_w = (int)cv->w;
    p.conv_c = (int)cv->c;
  }
  p.acc_f16 = acc_f16 ? 1 : 0;
  if (dq) {
    p.dequant = 1;
    p.relu = dq->relu;
    p.row_scale = dq->row_scale;
    p.bias = dq->bias;
    p.out_inv_scale = dq->out_inv_scale;
  }
  p.M = d->M; p.N = d->N; p.K = d->K;
  p.ldc = d->ldc; p.ldd = d->ldd;
  p.C = has_c ? C : nullptr;
  p.D = D;
  p.status = static_cast<uint32_t*>(workspace);
  p.alpha = falpha; p.beta = fbeta;
  p.a_fmt = (d->ab_type == SP24_BF16 || d->ab_type == SP24_E5M2) ? 1 : 0;
  p.cd_type = (int)d->cd_type;
  p.has_c = has_c ? 1 : 0;
  p.wait_limit = kWaitTimeoutCycles;
  // Test hooks for the failure path (set through sp24_test_set_fault_hooks only): a shorter limit, and a
  // pipeline that stalls by leaving out one k-block.  Nothing faults or hangs: the waits expire and the
  // kernel returns.
  Settings& cfg = settings();
  {
    const long long v = cfg.test_wait_cycles.load(std::memory_order_relaxed);
    if (v >= 1000000) p.wait_limit = v;
    p.test_skip_stage = cfg.test_skip_stage.load(std::memory_order_relaxed);
  }
  p.cd_col_major = d->order_d == SP24_COL_MAJOR ? 1 : 0;
  const bool sparse = !d->a_is_dense;
  const bool i8 = d->ab_type == SP24_I8, tf32 = d->ab_type == SP24_F32, f8 = is_fp8(d->ab_type);
  int ctas, block_n, mblk;
  choose_tile(d, ctas, block_n, mblk);
  p.band = 16 / mblk;
  if (const int c = cfg.ctas.load(std::memory_order_relaxed)) {
    ctas = c;
    block_n = cfg.block_n.load(std::memory_order_relaxed);
    mblk = cfg.mblk.load(std::memory_order_relaxed);
  }
  if (const int b = cfg.band.load(std::memory_order_relaxed)) p.band = b;
  const bool b_mn = d->order_b == SP24_ROW_MAJOR;  // B stored N-contiguous
  if (cfg.log.load(std::memory_order_relaxed))
    fprintf(stderr, "sp24_gemm: M=%lld N=%lld K=%lld ab=%d cd=%d %s%s tile=%dx%dx%d band=%d beta=%g%s%s\n", (long long)d->M,
            (long long)d->N, (long long)d->K, (int)d->ab_type, (int)d->cd_type, sparse ? "sparse" : "dense",
            b_mn ? " B:N-contiguous" : "", ctas, block_n, mblk, p.band, (double)fbeta, dq ? " dequant" : "",
            cv ? " conv3x3" : (acc_f16 ? " fp16-accumulate" : ""));
#define SP24_LAUNCH(K_, BN, CT, MB, MN)                                                               \
  (sparse ? launch<K_, true, BN, CT, MB, MN>(d, p, A, meta, B, s) : launch<K_, false, BN, CT, MB, MN>(d, p, A, meta, B, s))
#define SP24_DISPATCH(CT, BN, MB)                                                                     \
  if (ctas == CT && block_n == BN && mblk == MB && !b_mn && !tf32 && !f8) return i8 ? SP24_LAUNCH(1, BN, CT, MB, false) : SP24_LAUNCH(0, BN, CT, MB, false);
#define SP24_DISPATCH_TF32(CT, BN, MB)                                                                \
  if (ctas == CT && block_n == BN && mblk == MB && !b_mn && tf32) return SP24_LAUNCH(2, BN, CT, MB, false);
#define SP24_DISPATCH_F8(CT, BN, MB)                                                                  \
  if (ctas == CT && block_n == BN && mblk == MB && !b_mn && f8) return SP24_LAUNCH(3, BN, CT, MB, false);
#define SP24_DISPATCH_MN(CT, BN, MB)                                                                  \
  if (ctas == CT && block_n == BN && mblk == MB && b_mn)                                              \
    return tf32 ? SP24_LAUNCH(2, BN, CT, MB, true)                                                    \
                : (f8 ? SP24_LAUNCH(3, BN, CT, MB, true) : (i8 ? SP24_LAUNCH(1, BN, CT, MB, true) : SP24_LAUNCH(0, BN, CT, MB, true)));
  SP24_DISPATCH(1, 128, 1)
  SP24_DISPATCH(2, 224, 1)
  SP24_DISPATCH(2, 224, 2)
  SP24_DISPATCH(2, 192, 2)
  SP24_DISPATCH(2, 256, 1)
  if (ctas == 2 && block_n == 256 && mblk == 2 && !sparse && !b_mn && !tf32)  // dense variant only
    return f8 ? launch<3, false, 256, 2, 2, false>(d, p, A, meta, B, s)
              : (i8 ? launch<1, false, 256, 2, 2, false>(d, p, A, meta, B, s) : launch<0, false, 256, 2, 2, false>(d, p, A, meta, B, s));
  if (ctas == 2 && block_n == 240 && mblk == 1 && !b_mn && !tf32 && !f8 && !i8 && !p.cd_col_major && elem_bytes(d->cd_type) == 2)
    return SP24_LAUNCH(0, 240, 2, 1, false);
  SP24_DISPATCH_TF32(1, 128, 1)
  SP24_DISPATCH_TF32(2, 224, 1)
  SP24_DISPATCH_TF32(2, 224, 2)
  SP24_DISPATCH_TF32(2, 256, 1)
  SP24_DISPATCH_F8(1, 128, 1)
  SP24_DISPATCH_F8(2, 224, 1)
  SP24_DISPATCH_F8(2, 224, 2)
  SP24_DISPATCH_F8(2, 256, 1)
  SP24_DISPATCH_MN(1, 128, 1)
  SP24_DISPATCH_MN(2, 224, 1)
  SP24_DISPATCH_MN(2, 224, 2)
#undef SP24_DISPATCH
#undef SP24_DISPATCH_MN
#undef SP24_DISPATCH_TF32
#undef SP24_DISPATCH_F8
#undef SP24_LAUNCH
  return SP24_ERR_UNSUPPORTED;
}

extern "C" sp24_status sp24_gemm(const sp24_gemm_desc* d, const void* alpha, const void* A, const void* meta,
                                 const void* B, const void* beta, const void* C, void* D, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  return run_gemm(d, alpha, A, meta, B, beta, C, D, workspace, workspace_bytes, stream, nullptr);
}

extern "C" sp24_status sp24_gemm_f16acc(const sp24_gemm_desc* d, const void* alpha, const void* A, const void* meta,
                                        const void* B, const void* beta, const void* C, void* D, void* workspace,
                                        size_t workspace_bytes, void* stream) {
  SP24_RETURN_IF(d == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(d->ab_type != SP24_F16 || (d->cd_type != SP24_F16 && d->cd_type != SP24_F32), SP24_ERR_DTYPE);
  return run_gemm(d, alpha, A, meta, B, beta, C, D, workspace, workspace_bytes, stream, nullptr, nullptr, true);
}

extern "C" sp24_status sp24_gemm_i8_dequant(const sp24_gemm_desc* d, const void* A, const void* meta, const void* B,
                                            const float* row_scale, const float* bias, int relu, float out_scale,
                                            void* D, void* workspace, size_t workspace_bytes, void* stream) {
  SP24_RETURN_IF(d == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(d->M > 0 && d->N > 0 && row_scale == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(d->cd_type == SP24_I8 && !(out_scale > 0.f), SP24_ERR_UNSUPPORTED);
  DequantArgs dq = {row_scale, bias, relu ? 1 : 0, d->cd_type == SP24_I8 ? 1.0f / out_scale : 1.0f};
  return run_gemm(d, nullptr, A, meta, B, nullptr, nullptr, D, workspace, workspace_bytes, stream, &dq);
}

extern "C" sp24_status sp24_conv3x3_nhwc(const sp24_gemm_desc* d, int64_t Nb, int64_t H, int64_t W, int64_t Cin,
                                         const void* alpha, const void* A, const void* meta, const void* x,
                                         const void* beta, const void* C, void* D, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  SP24_RETURN_IF(d == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(Nb <= 0 || H <= 0 || W <= 0 || Cin <= 0, SP24_ERR_SHAPE);
  SP24_RETURN_IF(d->N != Nb * H * W || d->K != 9 * Cin, SP24_ERR_SHAPE);
  SP24_RETURN_IF(!is_ab_type(d->ab_type), SP24_ERR_DTYPE);
  // a shared-memory stage holds 128 (16-bit) or 256 (int8) consecutive k = channels of ONE filter tap
  const int64_t per_stage = elem_bytes(d->ab_type) == 1 ? 256 : 128;
  SP24_RETURN_IF(Cin % per_stage != 0, SP24_ERR_SHAPE);
  SP24_RETURN_IF(H > 32767 || W > 32767 || Nb > (int64_t(1) << 30), SP24_ERR_SHAPE);
  SP24_RETURN_IF(d->order_b != SP24_COL_MAJOR, SP24_ERR_UNSUPPORTED);
  // smaller activations trip a tensor-map restriction of current drivers
  SP24_RETURN_IF(Nb * H * W * Cin * elem_bytes(d->ab_type) < 131072, SP24_ERR_UNSUPPORTED);
  sp24_gemm_desc dd = *d;
  dd.ldb = d->K;  // not used by the im2col view, but keeps the generic checks meaningful
  ConvArgs cv = {Nb, H, W, Cin};
  return run_gemm(&dd, alpha, A, meta, x, beta, C, D, workspace, workspace_bytes, stream, nullptr, &cv);
}

extern "C" sp24_status sp24_gemm_status(void* workspace, void* stream) {
  SP24_RETURN_IF(workspace == nullptr, SP24_ERR_NULL);
  uint32_t host[4] = {0, 0, 0, 0};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  SP24_CUDA_CHECK(cudaMemcpyAsync(host, workspace, sizeof(host), cudaMemcpyDeviceToHost, s));
  SP24_CUDA_CHECK(cudaStreamSynchronize(s));
  if (host[0] == 0) return SP24_OK;
  // reported once: the record starts again from "ok" for the launches that follow
  SP24_CUDA_CHECK(cudaMemsetAsync(workspace, 0, sizeof(host), s));
  return SP24_ERR_TIMEOUT;
}

extern "C" sp24_status sp24_set_tile_override(int ctas, int block_n, int mblk, int band) {
  SP24_RETURN_IF(ctas < 0 || block_n < 0 || mblk < 0 || band < 0, SP24_ERR_SHAPE);
  Settings& cfg = settings();
  cfg.block_n.store(ctas ? block_n : 0, std::memory_order_relaxed);
  cfg.mblk.store(ctas ? (mblk ? mblk : 1) : 0, std::memory_order_relaxed);
  cfg.ctas.store(ctas, std::memory_order_relaxed);
  cfg.band.store(band, std::memory_order_relaxed);
  return SP24_OK;
}

extern "C" sp24_status sp24_test_set_fault_hooks(long long wait_cycles, int skip_stage) {
  Settings& cfg = settings();
  cfg.test_wait_cycles.store(wait_cycles, std::memory_order_relaxed);
  cfg.test_skip_stage.store(skip_stage ? 1 : 0, std::memory_order_relaxed);
  return SP24_OK;
}

// ---------------------------------------------------------------------------------------------
// sp24_gemm_static_ws: sp24_gemm for callers that cannot allocate device memory.
//
// sp24_gemm needs a small device workspace (its status record) that the caller normally
// allocates.  Some callers cannot: a serving process whose framework allocator has already
// reserved all device memory (cudaMalloc then fails), or a latency-critical loop that must not
// pay cudaMalloc's implicit device-wide synchronisation.  For them the workspace lives in the
// file-scope device array below, which every GPU that loads this library holds until the
// process exits.  Inputs and outputs are still the caller's.
//
// The array's name is only a host-side stand-in in host code, not a device address, so the
// address is resolved with cudaGetSymbolAddress once per device (with that device current) on
// the first call made on that device; that first call should therefore come before any stream
// capture.  The entry points call no cudaMalloc, cudaFree or other allocating routine.
//
// All calls on a device share the one array.  It starts out zero-filled (static storage) and the
// kernels only ever write a non-zero code into it, so nothing has to be cleared between calls:
// the record keeps the first expired wait of any call until sp24_gemm_static_ws_status reads and
// clears it.  Calls that overlap on the GPU (different streams) share that one record, so a
// reported timeout cannot be attributed to one of them: serialise them, or use sp24_gemm with
// one workspace per stream.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr size_t kStaticWorkspaceBytes = 4096;  // stated maximum; sp24_gemm currently needs 256
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_ws_mutex;
void* g_static_ws_ptr[kMaxDevices] = {};

// device address of the array on the current device (looked up once per device)
sp24_status static_workspace(void** out) {
  int dev = 0;
  SP24_CUDA_CHECK(cudaGetDevice(&dev));
  SP24_RETURN_IF(dev < 0 || dev >= kMaxDevices, SP24_ERR_UNSUPPORTED);
  std::lock_guard<std::mutex> lock(g_static_ws_mutex);
  if (g_static_ws_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || ptr == nullptr) return SP24_ERR_CUDA;
    g_static_ws_ptr[dev] = ptr;
  }
  *out = g_static_ws_ptr[dev];
  return SP24_OK;
}
}  // namespace

extern "C" sp24_status sp24_gemm_static_ws(const sp24_gemm_desc* d, const void* alpha, const void* A,
                                           const void* meta, const void* B, const void* beta, const void* C,
                                           void* D, void* stream) {
  SP24_RETURN_IF(d == nullptr, SP24_ERR_NULL);
  // the problem's workspace need must fit the fixed array
  SP24_RETURN_IF(sp24_gemm_workspace_bytes(d) > kStaticWorkspaceBytes, SP24_ERR_WORKSPACE);
  void* ws = nullptr;
  sp24_status st = static_workspace(&ws);
  if (st != SP24_OK) return st;
  return sp24_gemm(d, alpha, A, meta, B, beta, C, D, ws, kStaticWorkspaceBytes, stream);
}

extern "C" sp24_status sp24_gemm_static_ws_status(void* stream) {
  void* ws = nullptr;
  sp24_status st = static_workspace(&ws);
  if (st != SP24_OK) return st;
  return sp24_gemm_status(ws, stream);
}
