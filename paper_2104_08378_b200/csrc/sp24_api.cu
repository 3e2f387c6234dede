// Size helpers, status strings, the architecture check and the host-buffer pipeline.
#include "sp24_common.cuh"

namespace sp24 {

sp24_status check_arch() {
  static int cached_dev = -1;
  static sp24_status cached = SP24_ERR_ARCH;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SP24_ERR_CUDA;
  if (dev == cached_dev) return cached;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SP24_ERR_CUDA;
  cached_dev = dev;
  cached = major == 10 ? SP24_OK : SP24_ERR_ARCH;
  return cached;
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

extern "C" sp24_status sp24_pipeline_host(const sp24_gemm_desc* d, const void* alpha, const void* h_A, const void* h_B,
                                          const void* beta, const void* h_C, void* h_D, void* d_A, void* d_vals,
                                          void* d_meta, void* d_B, void* d_C, void* d_D, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  SP24_RETURN_IF(d == nullptr || alpha == nullptr || beta == nullptr, SP24_ERR_NULL);
  SP24_RETURN_IF(!is_ab_type(d->ab_type), SP24_ERR_DTYPE);
  SP24_RETURN_IF(d->a_is_dense, SP24_ERR_UNSUPPORTED);
  SP24_RETURN_IF(h_A == nullptr || h_B == nullptr || h_D == nullptr || d_A == nullptr || d_vals == nullptr ||
                     d_meta == nullptr || d_B == nullptr || d_D == nullptr,
                 SP24_ERR_NULL);
  const bool fp = d->ab_type != SP24_I8;
  const bool has_c = fp ? *static_cast<const float*>(beta) != 0.f : *static_cast<const int32_t*>(beta) != 0;
  SP24_RETURN_IF(has_c && (h_C == nullptr || d_C == nullptr), SP24_ERR_NULL);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t es = elem_bytes(d->ab_type), cs = elem_bytes(d->cd_type);
  SP24_CUDA_CHECK(cudaMemcpyAsync(d_A, h_A, (size_t)d->M * d->K * es, cudaMemcpyHostToDevice, s));
  SP24_CUDA_CHECK(cudaMemcpyAsync(d_B, h_B, (size_t)d->N * d->K * es, cudaMemcpyHostToDevice, s));
  if (has_c) SP24_CUDA_CHECK(cudaMemcpyAsync(d_C, h_C, (size_t)d->M * d->N * cs, cudaMemcpyHostToDevice, s));
  sp24_status st = sp24_compress(d->ab_type, d->M, d->K, d_A, d->K, d_vals, d->K / 2, d_meta, SP24_META_TCGEN05,
                                 nullptr, stream);
  if (st != SP24_OK) return st;
  sp24_gemm_desc packed = *d;
  packed.lda = d->K / 2;
  packed.ldb = d->K;
  packed.ldc = d->N;
  packed.ldd = d->N;
  st = sp24_gemm(&packed, alpha, d_vals, d_meta, d_B, beta, has_c ? d_C : nullptr, d_D, workspace, workspace_bytes,
                 stream);
  if (st != SP24_OK) return st;
  SP24_CUDA_CHECK(cudaMemcpyAsync(h_D, d_D, (size_t)d->M * d->N * cs, cudaMemcpyDeviceToHost, s));
  return SP24_OK;
}
