/*
 * sp24 -- 2:4 fine-grained structured-sparse matrix multiply for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library built from paper_2104_08378_b200/csrc.  The operations are the ones
 * "Accelerating Sparse Deep Neural Networks" (arXiv 2104.08378) defines:
 *
 *   - the 2:4 pattern: in every aligned group of four consecutive values along a row at
 *     least two are zero (Section 3, Section 3.1);
 *   - magnitude pruning: the two smallest-magnitude values of each group of four are removed
 *     (Section 4.1, step 2 of the workflow, Figure 5);
 *   - the compressed format: an R x C matrix is stored as R x C/2 kept values plus 2 bits of
 *     position metadata per kept value; a group with more than two zeros still stores two
 *     values (Section 3.1, Figure 1);
 *   - the sparse GEMM: sparse(M x K, stored M x K/2 + metadata) times dense(K x N) gives
 *     dense(M x N); B and C are dense (Section 3.2, Figure 2);
 *   - operand types FP16, BF16 (FP32 accumulate) and INT8 (INT32 accumulate) (Section 3.2,
 *     Table 1); dimensions are multiples of 16 for 16-bit and 32 for 8-bit types (Section 3.2).
 *
 * Conventions that hold for every entry point unless its comment says otherwise:
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library allocates no
 *     device memory and frees none.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work; they do not synchronise.
 *   - Argument errors are detected on the host, returned at once, and launch nothing.
 *   - Matrices are addressed as  element(i, j) = base[i * ld + j]  for ROW_MAJOR and
 *     base[j * ld + i] for COL_MAJOR; `ld` is in ELEMENTS.
 *   - A (the sparse operand) is always row-major with K contiguous, because the groups of
 *     four run along a row (Figure 1).
 *   - The device must be compute capability 10.0 (B200); anything else gives SP24_ERR_ARCH.
 *     There is no CPU fallback.
 */
#ifndef SP24_H_
#define SP24_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SP24_OK = 0,
  SP24_ERR_NULL = 1,        /* a required pointer is NULL                                  */
  SP24_ERR_DTYPE = 2,       /* dtype (or dtype combination) not supported by this call     */
  SP24_ERR_SHAPE = 3,       /* a dimension is negative or breaks the multiple-of rule      */
  SP24_ERR_STRIDE = 4,      /* a leading dimension is too small or not 16-byte granular    */
  SP24_ERR_ALIGN = 5,       /* a base pointer is not 16-byte aligned                       */
  SP24_ERR_UNSUPPORTED = 6, /* valid request outside what is built (e.g. int8 alpha != 1)  */
  SP24_ERR_WORKSPACE = 7,   /* workspace missing or smaller than sp24_gemm_workspace_bytes */
  SP24_ERR_CUDA = 8,        /* a CUDA runtime / driver call failed                         */
  SP24_ERR_TIMEOUT = 9,     /* a bounded device-side wait expired (see sp24_gemm_status)   */
  SP24_ERR_ARCH = 10        /* current device is not sm_100                                */
} sp24_status;

/* SP24_F32 as an OPERAND type selects the TF32 mode (Section 3.2, Table 1): FP32 storage, TF32
 * multiplication, FP32 accumulation, and the 1:2 pattern -- one kept value in every aligned
 * PAIR along K instead of two in every group of four.
 * SP24_E4M3 / SP24_E5M2 are the 8-bit floating-point encodings (1-4-3 without infinities, and
 * 1-5-2).  Table 1 of the paper has no 8-bit floating-point row (its hardware had none); they
 * use the 2:4 pattern and the format of the 8-bit integer row, with FP32 accumulation. */
typedef enum {
  SP24_F16 = 0, SP24_BF16 = 1, SP24_I8 = 2, SP24_F32 = 3, SP24_I32 = 4, SP24_E4M3 = 5, SP24_E5M2 = 6
} sp24_dtype;

/* Metadata layouts.
 * CANONICAL: row i occupies K/8 bytes starting at meta + i*K/8; group g of the row (columns
 *   4g..4g+3) owns bits 4g..4g+3 of that row's little-endian bit string; the nibble is
 *   p0 | (p1 << 2) with p0 < p1 the 0-based positions of the two kept values (Section 3.1:
 *   the example row with indices [[0,3],[1,2]] gives nibbles 0xC, 0x9, first byte 0x9C).
 * TCGEN05: the same nibbles permuted into the order the sm_100a sparse tensor-core
 *   instruction reads them from tensor memory, in 2048-byte blocks of 128 rows x 128 columns
 *   of A, rows padded to a multiple of 128 and K to a multiple of 256; padding nibbles are 0x4.
 *   This is the layout sp24_gemm consumes.
 * SP24_F32 (1:2 pattern): one nibble per PAIR, 0x4 if the first value of the pair is kept, 0xE if
 *   the second (the pair read as four 16-bit halves of which halves 0,1 or 2,3 survive).
 *   CANONICAL: K/4 bytes per row.  TCGEN05: the placement of the 16-bit types with a nibble
 *   standing for a pair: 2048-byte blocks of 128 rows x 64 columns, K padded to 128. */
typedef enum { SP24_META_CANONICAL = 0, SP24_META_TCGEN05 = 1 } sp24_meta_layout;

/* Which index of a matrix is contiguous in memory. */
typedef enum { SP24_ROW_MAJOR = 0, SP24_COL_MAJOR = 1 } sp24_order;

/* Human-readable name of a status code (static storage, never NULL). */
const char* sp24_status_string(sp24_status s);

/* Bytes of the kept-value array of an M x K matrix: M * (K/2) * sizeof(t)  (Figure 1:
 * R x C becomes R x C/2).  Returns 0 for an unsupported dtype or K % 4 != 0. */
size_t sp24_values_bytes(sp24_dtype t, int64_t M, int64_t K);

/* Bytes of the metadata of an M x K matrix.  CANONICAL: M*K/8 (2 bits per kept value,
 * Section 3.1, i.e. 12.5 % / 25 % of the kept values for 16-bit / 8-bit types).
 * TCGEN05: ceil(M/128) * ceil(K/256) * 4096.  Returns 0 for bad arguments. */
size_t sp24_meta_bytes(sp24_dtype t, int64_t M, int64_t K, sp24_meta_layout l);

/* Magnitude pruning to 2:4 (Section 4.1 step 2; pattern of Section 3).
 * For every row i < M and every aligned group of four columns 4g..4g+3 < K the two values of
 * largest magnitude are copied bit-for-bit to y, the other two positions receive +0.  Equal
 * magnitudes: the lower column index is kept.  Magnitude is |x| for I8 (so -128 ranks as
 * 128) and the bit pattern without its sign bit for F16/BF16/E4M3/E5M2 (denormals are not
 * flushed).
 *   t: SP24_F16, SP24_BF16, SP24_I8, SP24_E4M3 or SP24_E5M2.   M >= 0, K >= 0, K % 4 == 0.
 *      SP24_F32: the 1:2 pattern -- the larger magnitude of every aligned pair is kept, equal
 *      magnitudes keep the first (K % 8 == 0, 16-byte aligned pointers and rows required;
 *      the same holds for sp24_compress / sp24_decompress, whose vals are then M x K/2 FP32).
 *   x: device, M x K row-major, leading dimension ldx >= K (elements).
 *   y: device, same shape, leading dimension ldy >= K; may be the same buffer as x.
 * Fastest when x, y are 16-byte aligned and ldx*sizeof(t), ldy*sizeof(t), K*sizeof(t) are
 * multiples of 16; other cases take a scalar path with the same result. */
sp24_status sp24_prune(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx,
                       void* y, int64_t ldy, void* stream);

/* Compression to kept values + metadata (Section 3.1, Figure 1).
 * Applies the selection rule of sp24_prune to x itself, so compress(x) == compress(prune(x))
 * and the call doubles as the fused prune+compress pass.  For group g of row i with kept
 * positions p0 < p1:  vals[i*ldv + 2g] = x[i, 4g+p0],  vals[i*ldv + 2g+1] = x[i, 4g+p1],
 * metadata nibble p0 | (p1<<2) stored as `l` says.  A group with fewer than two non-zeros is
 * completed with its lowest-index zeros (an all-zero group stores positions 0,1).
 *   vals: device, M x K/2 row-major, ldv >= K/2 (elements).
 *   meta: device, sp24_meta_bytes(t, M, K, l) bytes; for TCGEN05 the padding is written too.
 *   dropped_nonzeros: device counter or NULL.  If given, the number of non-kept positions
 *     holding a non-zero magnitude is ADDED to it (0 added iff x already was 2:4).
 * Requires K % 4 == 0 (K % 16 == 0 for the vectorised path). */
sp24_status sp24_compress(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx,
                          void* vals, int64_t ldv, void* meta, sp24_meta_layout l,
                          unsigned long long* dropped_nonzeros, void* stream);

/* sp24_prune and sp24_compress in ONE pass over x (Section 4.1 step 2 followed by the storage
 * format of Section 3.1): y receives what sp24_prune(x) would write, vals / meta / dropped what
 * sp24_compress(x) would, bit for bit; x is read once instead of twice and the pruned matrix is
 * not re-read.  Arguments as for the two calls; y may be the same buffer as x.  Operands the
 * vectorised kernels cannot take (see sp24_prune) and the SP24_F32 1:2 pattern run as the two
 * separate passes. */
sp24_status sp24_prune_compress(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx,
                                void* y, int64_t ldy, void* vals, int64_t ldv, void* meta,
                                sp24_meta_layout l, unsigned long long* dropped_nonzeros,
                                void* stream);

/* Inverse of sp24_compress (the metadata is what decodes the format, Section 3.1):
 * y is M x K row-major (ldy >= K) with y[i, 4g+p_t] = vals[i, 2g+t] and +0 elsewhere. */
sp24_status sp24_decompress(sp24_dtype t, int64_t M, int64_t K, const void* vals, int64_t ldv,
                            const void* meta, sp24_meta_layout l, void* y, int64_t ldy,
                            void* stream);

/* Problem description of D = alpha * op(A) * B + beta * C  (Section 3.2, Figure 2).
 *   ab_type: SP24_F16 or SP24_BF16 (FP32 accumulate), SP24_I8 (INT32 accumulate) or SP24_F32
 *            (TF32 mode, 1:2 pattern, FP32 accumulate; cd_type SP24_F32 only; inputs are used
 *            with their low 13 mantissa bits ignored) -- the operand/accumulator pairs of
 *            Table 1 (its FP16-accumulate row is sp24_gemm_f16acc).  SP24_E4M3 or SP24_E5M2
 *            (both operands the same type, FP32 accumulate) go beyond that table.
 *   cd_type: type of C and D.  F16/BF16 operands: SP24_F16, SP24_BF16 (ab_type's own) or
 *            SP24_F32.  I8 operands: SP24_I32.  E4M3/E5M2 operands: SP24_F16, SP24_BF16 or
 *            SP24_F32.
 *   M, N, K: K is the LOGICAL (uncompressed) reduction length.  M, N, K must be multiples of
 *            16 (16-bit types) or 32 (8-bit types) (Section 3.2); zero-sized problems return
 *            SP24_OK.
 *   lda:     leading dimension of the A-side value array: of vals (M x K/2) when
 *            a_is_dense == 0, of the dense M x K matrix when a_is_dense == 1.
 *   order_b: SP24_COL_MAJOR = K contiguous (B stored as N rows of K values: the
 *            [tokens, hidden] activation layout; ldb >= K), the faster order, or
 *            SP24_ROW_MAJOR = N contiguous (the K x N matrix stored row by row; ldb >= N).
 *   order_c / order_d: SP24_ROW_MAJOR (N contiguous; ldc, ldd >= N) or SP24_COL_MAJOR
 *            (M contiguous, the [tokens, out_features] layout; ldc, ldd >= M).  When C is
 *            used (beta != 0) it must have the same order as D.
 *   a_is_dense: 0 = 2:4 compressed A with TCGEN05 metadata (the sparse tensor-core path);
 *            1 = the dense variant on the same pipeline (`A` is M x K dense, `meta` unused).
 * All leading dimensions are in elements and, in bytes, multiples of 16. */
typedef struct {
  sp24_dtype ab_type, cd_type;
  int64_t M, N, K;
  int64_t lda, ldb, ldc, ldd;
  sp24_order order_b, order_c, order_d;
  int a_is_dense;
} sp24_gemm_desc;

/* Reports the tile shape sp24_gemm (and its variants) would use for this problem on the current
 * device: CTAs per tile (1, or 2 = a pair working on one tile), columns per tile, 128-row blocks
 * per CTA.  The output tile is (128 * ctas * mblk) x block_n.  Launches nothing. */
sp24_status sp24_gemm_plan(const sp24_gemm_desc* d, int* ctas, int* block_n, int* mblk);

/* Bytes of device workspace sp24_gemm needs for this problem (currently a fixed 256 bytes:
 * the device-side status record).  The workspace must be 16-byte aligned. */
size_t sp24_gemm_workspace_bytes(const sp24_gemm_desc* d);

/* The 2:4 sparse GEMM on the sparse tensor cores (Section 3.2, Figure 2):
 *   D[i,j] = alpha * sum_g sum_{t=0,1} vals[i,2g+t] * B[4g + p_t(i,g), j] + beta * C[i,j].
 *   alpha, beta: HOST pointers.  float for floating-point operands; int32_t for I8, where only
 *                alpha == 1 and beta in {0, 1} are built (else SP24_ERR_UNSUPPORTED).
 *   A:    device; vals (M x K/2) or dense A (M x K), row-major, 16-byte aligned.
 *   meta: device; TCGEN05-layout metadata of A (ignored when a_is_dense).
 *   B, C, D: device, 16-byte aligned.  C may be NULL iff beta == 0.  C may alias D.
 *   workspace: device, >= sp24_gemm_workspace_bytes(d), zero-filled before its first use.  The
 *              kernel records an expired wait there; see sp24_gemm_status.
 * Accumulation is FP32 (INT32) in hardware order; the result is rounded to cd_type once,
 * round-to-nearest-even.
 * The tile shape is chosen from the problem size (sp24_set_tile_override forces one).
 * The five tensor maps of a call are kept in a small per-thread host cache keyed by address,
 * shape and leading dimension, so repeated calls on the same buffers do not encode them again. */
sp24_status sp24_gemm(const sp24_gemm_desc* d, const void* alpha, const void* A,
                      const void* meta, const void* B, const void* beta, const void* C,
                      void* D, void* workspace, size_t workspace_bytes, void* stream);

/* The FP16-accumulation mode of Table 1 (FP16 operands, FP16 accumulator; Section 3.2): sp24_gemm
 * with the tensor cores adding the products into a binary16 accumulator instead of an FP32 one.
 *   d->ab_type must be SP24_F16; d->cd_type SP24_F16 or SP24_F32; everything else as for sp24_gemm
 *   (sparse or dense variant, both orders of B, C and D; alpha, beta and C are applied in FP32 to
 *   the widened accumulator).
 * Accuracy: the running sum is rounded to binary16 after every tensor-core instruction (32 values of
 * K for the sparse form, 16 for the dense one), so the error grows with K:
 * |err| <= (K/32 + 2) * 2^-10 * (|A|.|B|)_ij is the bound the tests use, against 2^-11 relative for
 * one final rounding with sp24_gemm.  On these tensor cores a binary16 accumulator occupies a full
 * 32-bit cell of tensor memory and the instruction rate is that of FP32 accumulation, so the mode
 * buys no speed here (measured; see the benchmark's other_configs): it exists for bit-compatibility
 * with deployments that used it. */
sp24_status sp24_gemm_f16acc(const sp24_gemm_desc* d, const void* alpha, const void* A,
                             const void* meta, const void* B, const void* beta, const void* C,
                             void* D, void* workspace, size_t workspace_bytes, void* stream);

/* INT8 sparse GEMM with a dequantising epilogue, for the deployment the paper describes in
 * Section 4.4 and Section 5.1: INT8 weights and activations, per-row scaling factors for the
 * weights of fully-connected layers and a per-tensor factor for the activations.
 *   D[i,j] = act( row_scale[i] * acc[i,j] + bias[i] ),   acc = INT32 result of the 2:4 product,
 * where row_scale[i] is the caller's product of the weight row's factor and the activation
 * tensor's factor, bias may be NULL (0) and act is the identity or max(., 0) (relu != 0).
 *   d->ab_type must be SP24_I8; d->cd_type: SP24_BF16, SP24_F16, SP24_F32, or SP24_I8.
 *   SP24_I8 output: q = round-to-nearest-even(D / out_scale) clamped to [-127, 127].
 *   row_scale, bias: device, M floats.  Everything is computed in FP32 in this order: acc to
 *   float, one fused multiply-add with scale and bias, the activation, one multiply by
 *   1/out_scale (rounded to float once on the host), the rounding.
 * Other arguments, layouts and the workspace are those of sp24_gemm (alpha, beta, C unused). */
sp24_status sp24_gemm_i8_dequant(const sp24_gemm_desc* d, const void* A, const void* meta,
                                 const void* B, const float* row_scale, const float* bias,
                                 int relu, float out_scale, void* D, void* workspace,
                                 size_t workspace_bytes, void* stream);

/* 3x3, stride-1, pad-1 convolution of an NHWC activation with 2:4-sparse weights as an implicit
 * GEMM (Section 4.2: a convolution's reduction dimension is C*R*S): the same kernel as sp24_gemm,
 * but the B operand is read straight from the activation by im2col-mode TMA loads instead of
 * from a materialised (Nb*H*W) x 9*Cin matrix.
 *   d:  as for sp24_gemm with N = Nb*H*W output pixels (pixel (n,h,w) is column (n*H+h)*W+w) and
 *       K = 9*Cin ordered (r, s, c), c fastest; d->M output channels; ldb ignored; order_b must
 *       be SP24_COL_MAJOR.  With order_d = SP24_COL_MAJOR the output is NHWC ([pixels, M]).
 *   x:  device, Nb x H x W x Cin, packed, 16-byte aligned, at least 128 KiB.
 *   Cin must be a multiple of 128 (16-bit types) or 256 (int8).
 *   A / meta / alpha / beta / C / D / workspace: as for sp24_gemm (a_is_dense selects the dense
 *   variant with A = Kout x 9*Cin). */
sp24_status sp24_conv3x3_nhwc(const sp24_gemm_desc* d, int64_t Nb, int64_t H, int64_t W, int64_t Cin,
                              const void* alpha, const void* A, const void* meta, const void* x,
                              const void* beta, const void* C, void* D, void* workspace,
                              size_t workspace_bytes, void* stream);

/* Reads the status record in `workspace` back to the host (synchronises `stream`) and returns
 * SP24_OK, or SP24_ERR_TIMEOUT if a bounded wait inside any GEMM kernel that used this workspace
 * since the last read expired (that kernel returned early and its D is incomplete).
 * The record is STICKY: `workspace` must be zero-filled once before its first use (e.g.
 * cudaMemsetAsync); the kernels never clear it, they only write the code of the first wait that
 * expired into word 0 and count expired waits in word 1.  One record therefore covers any number
 * of launches (a benchmark loop, the bands of sp24_pipeline_host): a timeout in any of them is
 * still there when this call reads it.  A reported timeout is cleared by this call (a memset on
 * `stream`), so that the next read concerns the launches that follow. */
sp24_status sp24_gemm_status(void* workspace, void* stream);

/* (No counterpart in the paper: a deployment variant of sp24_gemm.)
 * sp24_gemm for callers that cannot allocate device memory -- a process whose framework
 * allocator already owns all of the GPU's memory, so that cudaMalloc fails, or a serving loop
 * that cannot afford the device-wide synchronisation cudaMalloc implies.  The workspace
 * (status record) lives in a fixed 4096-byte device array inside the library, present on every
 * GPU that loads the library until the process exits; problems whose
 * sp24_gemm_workspace_bytes exceeds 4096 are refused with SP24_ERR_WORKSPACE.  Arguments and
 * results are those of sp24_gemm; inputs and outputs remain the caller's buffers.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress);
 * make that first call before any stream capture.  Nothing is allocated or freed.
 * All calls on a device share the array.  It starts zero-filled and nothing has to be cleared
 * between calls: the kernels only write into it when a bounded wait expires, and the record
 * then stays until sp24_gemm_static_ws_status reads it.  Two calls that overlap on the GPU
 * (different streams) share the one record, so a timeout cannot be attributed to one of them:
 * serialise such calls, or use sp24_gemm with a workspace per stream. */
sp24_status sp24_gemm_static_ws(const sp24_gemm_desc* d, const void* alpha, const void* A,
                                const void* meta, const void* B, const void* beta,
                                const void* C, void* D, void* stream);

/* (No counterpart in the paper.)  sp24_gemm_status for the array of sp24_gemm_static_ws on the
 * current device: synchronises `stream`, returns SP24_OK or SP24_ERR_TIMEOUT (and then clears
 * the record).  Allocates nothing. */
sp24_status sp24_gemm_static_ws_status(void* stream);

/* Benchmarking and test support (no counterpart in the paper): forces the tile shape of every
 * following sp24_gemm / sp24_gemm_i8_dequant / sp24_conv3x3_nhwc call in this process.
 *   ctas: 1 or 2 CTAs per tile; block_n: columns per tile; mblk: 128-row blocks per CTA (1 or 2);
 *   the shape must be one of the built ones, else those calls return SP24_ERR_UNSUPPORTED.
 *   ctas == 0 restores the automatic choice.  band: m-tiles per band of the tile sweep, 0 = default.
 * The environment variables SP24_TILE=<ctas>x<block_n>x<mblk>, SP24_BAND=<band> and SP24_LOG=1
 * (print the problem and the chosen tile shape of every call to stderr) give the initial values;
 * they are read ONCE, at the first GEMM call of the process. */
sp24_status sp24_set_tile_override(int ctas, int block_n, int mblk, int band);

/* Test support for the failure path, not for production use: shortens the limit of every
 * device-side wait to `wait_cycles` SM cycles (values below 1 000 000 restore the default of
 * about a second) and, with skip_stage != 0, makes the TMA producers leave out one k-block of
 * their first tile so that a wait expires.  Nothing faults or hangs: the kernel returns early
 * and sp24_gemm_status reports SP24_ERR_TIMEOUT.  Never read from the environment. */
sp24_status sp24_test_set_fault_hooks(long long wait_cycles, int skip_stage);

/* Lowering of a 3x3, stride-1, pad-1 NHWC convolution input to the GEMM's B operand
 * (Section 4.2: a convolution's reduction dimension is C*R*S).  Output is K-contiguous:
 *   out[((n*H + h)*W + w) * ldo + (r*3 + s)*C + c] = in[n, h+r-1, w+s-1, c]  (0 outside).
 *   t: SP24_F16, SP24_BF16, SP24_I8, SP24_E4M3 or SP24_E5M2.  C*sizeof(t) must be a multiple
 *   of 16; ldo >= 9*C. */
sp24_status sp24_im2col_nhwc_3x3(sp24_dtype t, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                 const void* in, void* out, int64_t ldo, void* stream);

/* Figure of merit of a channel permutation (Section 4.1: permuting the columns of the weight
 * matrix before pruning so that large values are spread over the groups keeps more total
 * magnitude).  Adds to *result (device double) the sum of |x[i, perm[k]]| over the positions
 * that 2:4 pruning of the column-permuted matrix x'[:, k] = x[:, perm[k]] keeps.
 *   perm: device, K int32 column indices (a permutation of 0..K-1), or NULL for the identity.
 *   t: SP24_F16, SP24_BF16, SP24_I8;  K % 4 == 0;  ldx >= K.  Summation is in double; the
 *   order of the partial sums is not fixed. */
sp24_status sp24_kept_magnitude(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx,
                                const int32_t* perm, double* result, void* stream);

/* Re-imposes a fixed 2:4 pattern on updated weights, as sparse retraining does (Section 4.1,
 * step 3: the pattern found in step 2 is kept while the weights train on):
 * y[i, k] = w[i, k] where the metadata of sp24_compress names k as kept, +0 elsewhere.
 *   meta / l: metadata of an M x K matrix in either layout.  K % 8 == 0; y may alias w. */
sp24_status sp24_apply_mask(sp24_dtype t, int64_t M, int64_t K, const void* w, int64_t ldw,
                            const void* meta, sp24_meta_layout l, void* y, int64_t ldy,
                            void* stream);

/* 2:4 along rows AND columns (Section 6: the pattern must also hold for the transposed weights
 * if the backward pass is to be accelerated).  Every aligned 4 x 4 block keeps exactly two
 * values per row and per column; of the 90 such patterns the one keeping the largest total
 * magnitude is taken (exhaustive search).  Score of a pattern: ((s0 + s1) + s2) + s3 with
 * s_i = |x[i, c]| + |x[i, c']| for the row's kept columns c < c', in FP32; patterns are numbered
 * lexicographically by their rows' kept pairs in the order 01, 02, 03, 12, 13, 23, and the
 * lowest-numbered pattern with the largest score wins.  M % 4 == 0, K % 4 == 0; y may alias x. */
sp24_status sp24_prune_2d(sp24_dtype t, int64_t M, int64_t K, const void* x, int64_t ldx,
                          void* y, int64_t ldy, void* stream);

/* End-to-end convenience for callers whose data lives in HOST memory (pinned for speed):
 * copies dense A (M x K, row-major, packed), B (N rows of K, packed) and, if beta != 0, C
 * (M x N packed) to the device buffers the caller provides, runs sp24_compress (TCGEN05
 * layout) and sp24_gemm, and copies D (M x N packed) back.  All h_* are host pointers, all
 * d_* device pointers sized for the packed matrices (d_vals, d_meta as the size helpers
 * say).  Work is enqueued on `stream`; the caller synchronises.  For M >= 16384 the work runs
 * in up to eight row bands: each band's D is copied out on a second, library-owned stream
 * (created once per device; `stream` is made to wait for it before the call returns) while
 * the next band's A and C are copied in, so both directions of the host link are busy.  The status
 * record in `workspace` is sticky (see sp24_gemm_status), so it covers every band.  The call may be
 * made from several host threads at once (events are created per call). */
sp24_status sp24_pipeline_host(const sp24_gemm_desc* d, const void* alpha, const void* h_A,
                               const void* h_B, const void* beta, const void* h_C, void* h_D,
                               void* d_A, void* d_vals, void* d_meta, void* d_B, void* d_C,
                               void* d_D, void* workspace, size_t workspace_bytes,
                               void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SP24_H_ */
