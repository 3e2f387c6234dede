// Size helpers, status strings, the architecture check and the host-buffer pipeline.
#include <atomic>
#include <mutex>

#include "sp24_common.cuh"

namespace sp24 {

sp24_status check_arch() {
  // per-device answer: 0 = not asked yet, 1 = sm_100, 2 = something else (callers may be on several threads)
  static std::atomic<int> known[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SP24_ERR_CUDA;
  const bool cacheable = dev >= 0 && dev < 64;
  if (cacheable) {
    const int k = known[dev].load(std::memory_order_relaxed);
    if (k != 0) return k == 1 ? SP24_OK : SP24_ERR_ARCH;
  }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SP24_ERR_CUDA;
  if (cacheable) known[dev].store(major == 10 ? 1 : 2, std::memory_order_relaxed);
  return major == 10 ? SP24_OK : SP24_ERR_ARCH;
}

}  // namespace sp24

using namespace sp24;

extern "C" const char* sp24_status_string(sp24_status s) {
  switch (s) {
    case SP24_OK: return "ok";
    case SP24_ERR_NULL: return "null pointer";
    case SP24_ERR_DTYPE: return "unsupported dtype";
    case SP24_ERR_SHAPE: return "bad shape";
    case SP24_ERR_STRIDE: return "bad leading dimension";
    case SP24_ERR_ALIGN: return "pointer not 16-byte aligned";
    case SP24_ERR_UNSUPPORTED: return "not built";
    case SP24_ERR_WORKSPACE: return "workspace missing or too small";
    case SP24_ERR_CUDA: return "CUDA call failed";
    case SP24_ERR_TIMEOUT: return "bounded device wait expired";
    case SP24_ERR_ARCH: return "device is not sm_100";
  }
  return "unknown status";
}

extern "C" size_t sp24_values_bytes(sp24_dtype t, int64_t M, int64_t K) {
  if (t == SP24_F32) return (M < 0 || K < 0 || K % 2 != 0) ? 0 : (size_t)M * (size_t)(K / 2) * 4;
  if (!is_ab_type(t) || M < 0 || K < 0 || K % 4 != 0) return 0;
  return (size_t)M * (size_t)(K / 2) * (size_t)elem_bytes(t);
}

extern "C" size_t sp24_meta_bytes(sp24_dtype t, int64_t M, int64_t K, sp24_meta_layout l) {
  if (t == SP24_F32) {  // 1:2 pattern: one nibble per pair
    if (M < 0 || K < 0 || K % 4 != 0) return 0;
    if (l == SP24_META_CANONICAL) return (size_t)M * (size_t)(K / 4);
    if (l == SP24_META_TCGEN05) return (size_t)((M + 127) / 128) * (size_t)((K + 127) / 128) * 4096;
    return 0;
  }
  if (!is_ab_type(t) || M < 0 || K < 0 || K % 8 != 0) return 0;
  if (l == SP24_META_CANONICAL) return (size_t)M * (size_t)(K / 8);
  if (l == SP24_META_TCGEN05) return (size_t)((M + 127) / 128) * (size_t)((K + 255) / 256) * 4096;
  return 0;
}

namespace {

// Second stream of the host-buffer pipeline, created once per device and kept (a stream holds no
// device memory).  It is shared by all callers; what orders one call's copies behind its own
// GEMMs are events, and those are created per call (see BandEvents), so calls from several host
// threads do not disturb one another.
constexpr int kMaxBands = 8;

sp24_status side_stream(cudaStream_t* out) {
  static std::mutex mu;
  static cudaStream_t per_device[64] = {};
  int dev = 0;
  SP24_CUDA_CHECK(cudaGetDevice(&dev));
  SP24_RETURN_IF(dev < 0 || dev >= 64, SP24_ERR_UNSUPPORTED);
  std::lock_guard<std::mutex> lock(mu);
  if (per_device[dev] == nullptr) SP24_CUDA_CHECK(cudaStreamCreateWithFlags(&per_device[dev], cudaStreamNonBlocking));
  *out = per_device[dev];
  return SP24_OK;
}

// The events of ONE sp24_pipeline_host call: one per band (GEMM done -> copy-out may start) and
// one for the final join.  Destroyed when the call returns; an event that is still pending is
// released by the runtime once it has completed.
struct BandEvents {
  cudaEvent_t band_done[kMaxBands] = {};
  cudaEvent_t joined = nullptr;
  sp24_status create(int bands) {
    for (int b = 0; b < bands; ++b) SP24_CUDA_CHECK(cudaEventCreateWithFlags(&band_done[b], cudaEventDisableTiming));
    SP24_CUDA_CHECK(cudaEventCreateWithFlags(&joined, cudaEventDisableTiming));
    return SP24_OK;
  }
  ~BandEvents() {
    for (cudaEvent_t e : band_done)
      if (e) cudaEventDestroy(e);
    if (joined) cudaEventDestroy(joined);
  }
};

}  // namespace

extern "C" sp24_status sp24_pipeline_host(const sp24_gemm_desc* d, const void* alpha, const void* h_A, const void* h_B,
                                          const void* beta, const void* h_C, void* h_D, void* d_A, void* d_vals,
                                          void* d_meta, void* d_B, void* d_C, void* d_D, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  SP24_RETURN_IF(d == nullptr || alpha == nullptr || beta == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(!is_ab_type(d->ab_type), SP24_ERR_DTYPE);
  SP24_RETURN_IF(d->a_is_dense, SP24_ERR_UNSUPPORTED);
  SP24_RETURN_IF(d->M < 0 || d->N < 0 || d->K <= 0, SP24_ERR_SHAPE);
  SP24_RETURN_IF(h_A == nullptr || h_B == nullptr || h_D == nullptr || d_A == nullptr || d_vals == nullptr ||
                     d_meta == nullptr || d_B == nullptr || d_D == nullptr,
                 SP24_ERR_NULL);
  const bool fp = d->ab_type != SP24_I8;
  const bool has_c = fp ? *static_cast<const float*>(beta) != 0.f : *static_cast<const int32_t*>(beta) != 0;
  SP24_RETURN_IF(has_c && (h_C == nullptr || d_C == nullptr), SP24_ERR_NULL);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t es = elem_bytes(d->ab_type), cs = elem_bytes(d->cd_type);
  SP24_RETURN_IF(cs == 0, SP24_ERR_DTYPE);
  SP24_CUDA_CHECK(cudaMemcpyAsync(d_B, h_B, (size_t)d->N * d->K * es, cudaMemcpyHostToDevice, s));
  sp24_status st = SP24_OK;
  // Row bands of A / C / D (multiples of the 512-row tile): the copy-out of one band runs on a
  // second stream while the caller's stream copies in the next band's A and C, compresses and
  // multiplies it, so the two directions of the host link work at the same time.
  int bands = (int)(d->M / 8192);
  bands = bands < 1 ? 1 : (bands > kMaxBands ? kMaxBands : bands);
  const int64_t band_rows = bands == 1 ? d->M : ((d->M + bands - 1) / bands + 511) / 512 * 512;
  cudaStream_t side = nullptr;
  BandEvents ev;
  if (bands > 1) {
    if ((st = side_stream(&side)) != SP24_OK) return st;
    if ((st = ev.create(bands)) != SP24_OK) return st;
  }
  const size_t meta_block_bytes = sp24_meta_bytes(d->ab_type, 128, d->K, SP24_META_TCGEN05);  // per 128 rows
  int issued = 0;
  // one band; any failure leaves through the join below, so that copies already queued on the
  // second stream are ordered before whatever the caller enqueues next
  auto run_band = [&](int b) -> sp24_status {
    const int64_t r0 = (int64_t)b * band_rows, r1 = r0 + band_rows < d->M ? r0 + band_rows : d->M;
    if (r0 >= r1) return SP24_OK;
    const size_t c_off = (size_t)r0 * d->N * cs, c_bytes = (size_t)(r1 - r0) * d->N * cs;
    const size_t a_off = (size_t)r0 * d->K * es, v_off = (size_t)r0 * (d->K / 2) * es;
    const size_t m_off = (size_t)(r0 / 128) * meta_block_bytes;
    SP24_CUDA_CHECK(cudaMemcpyAsync(static_cast<char*>(d_A) + a_off, static_cast<const char*>(h_A) + a_off,
                                    (size_t)(r1 - r0) * d->K * es, cudaMemcpyHostToDevice, s));
    sp24_status bs = sp24_compress(d->ab_type, r1 - r0, d->K, static_cast<const char*>(d_A) + a_off, d->K,
                                   static_cast<char*>(d_vals) + v_off, d->K / 2, static_cast<char*>(d_meta) + m_off,
                                   SP24_META_TCGEN05, nullptr, stream);
    if (bs != SP24_OK) return bs;
    if (has_c)
      SP24_CUDA_CHECK(cudaMemcpyAsync(static_cast<char*>(d_C) + c_off, static_cast<const char*>(h_C) + c_off, c_bytes,
                                      cudaMemcpyHostToDevice, s));
    sp24_gemm_desc packed = *d;
    packed.M = r1 - r0;
    packed.lda = d->K / 2;
    packed.ldb = d->K;
    packed.ldc = d->N;
    packed.ldd = d->N;
    bs = sp24_gemm(&packed, alpha, static_cast<const char*>(d_vals) + v_off, static_cast<const char*>(d_meta) + m_off,
                   d_B, beta, has_c ? static_cast<const char*>(d_C) + c_off : nullptr, static_cast<char*>(d_D) + c_off,
                   workspace, workspace_bytes, stream);
    if (bs != SP24_OK) return bs;
    cudaStream_t out = s;
    if (bands > 1) {
      SP24_CUDA_CHECK(cudaEventRecord(ev.band_done[b], s));
      SP24_CUDA_CHECK(cudaStreamWaitEvent(side, ev.band_done[b], 0));
      out = side;
      ++issued;
    }
    SP24_CUDA_CHECK(cudaMemcpyAsync(static_cast<char*>(h_D) + c_off, static_cast<const char*>(d_D) + c_off, c_bytes,
                                    cudaMemcpyDeviceToHost, out));
    return SP24_OK;
  };
  for (int b = 0; b < bands && st == SP24_OK; ++b) st = run_band(b);
  if (issued) {  // the caller's stream ends behind every copy made on the second one, also after a failure
    const bool joined = cudaEventRecord(ev.joined, side) == cudaSuccess && cudaStreamWaitEvent(s, ev.joined, 0) == cudaSuccess;
    if (!joined) {
      cudaStreamSynchronize(side);  // last resort: order by waiting on the host
      if (st == SP24_OK) st = SP24_ERR_CUDA;
    }
  }
  return st;
}
