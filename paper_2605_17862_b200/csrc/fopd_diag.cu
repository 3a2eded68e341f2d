// Diagnostic entry points: row-wise KL / entropy between two logit tensors, the
// supervision drift and alignment ratio per sample, and the buffer refresh rule.
#include "diag_kernels.cuh"
#include "host_common.cuh"

using namespace fopd;

extern "C" {

int fopd_row_divergence(const void *first, const void *second, const uint8_t *mask, const int32_t *sample_id,
                        int64_t n_rows, int64_t vocab, int64_t row_stride, int32_t dtype, int32_t B, float *kl,
                        float *entropy, double *acc, int32_t *status, void *stream) {
  if (dtype != FOPD_BF16 && dtype != FOPD_F32) return FOPD_ERR_DTYPE;
  if (n_rows < 0 || vocab <= 0 || row_stride < vocab || B <= 0 || vocab > (int64_t)1 << 30) return FOPD_ERR_SIZE;
  if (!acc) return FOPD_ERR_NULL;
  if (n_rows == 0) return FOPD_OK;
  if (!first || !second || !mask || !sample_id) return FOPD_ERR_NULL;
  const int64_t esz = dtype == FOPD_BF16 ? 2 : 4;
  if (!aligned16(first) || !aligned16(second) || (row_stride * esz) % 16 != 0) return FOPD_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // one temporary: the samples' row ranges, then {kl, entropy} of every row
  const size_t bb = (bounds_bytes(B) + 255) & ~size_t(255);
  char *tmp = nullptr;
  int rc = scratch_alloc(reinterpret_cast<void **>(&tmp), bb + (size_t)n_rows * sizeof(float2), st);
  if (rc != FOPD_OK) return rc;
  unsigned long long *bounds = reinterpret_cast<unsigned long long *>(tmp);
  float2 *vals = reinterpret_cast<float2 *>(tmp + bb);
  const unsigned grid = row_grid(n_rows);
  if (dtype == FOPD_BF16)
    row_divergence_kernel<FOPD_BF16><<<grid, kDiagThreads, 0, st>>>(first, second, mask, sample_id, n_rows, vocab,
                                                                  row_stride, B, kl, entropy, vals, status);
  else
    row_divergence_kernel<FOPD_F32><<<grid, kDiagThreads, 0, st>>>(first, second, mask, sample_id, n_rows, vocab,
                                                                 row_stride, B, kl, entropy, vals, status);
  rc = launch_ok();
  if (rc == FOPD_OK) rc = launch_sample_bounds(sample_id, n_rows, B, bounds, st);
  if (rc == FOPD_OK) {
    divergence_reduce_kernel<<<B, kSegThreads, 0, st>>>(sample_id, mask, n_rows, vals, bounds_or_null(bounds, B), acc);
    rc = launch_ok();
  }
  if (cudaFreeAsync(tmp, st) != cudaSuccess) rc = FOPD_ERR_CUDA;
  return rc;
}

int fopd_supervision_drift(const double *acc, const int32_t *seq_len, int32_t B, float *d_sup, float *m_sup,
                           float *mean_entropy, void *stream) {
  if (B <= 0) return FOPD_ERR_SIZE;
  if (!acc || !seq_len) return FOPD_ERR_NULL;
  supervision_drift_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(acc, seq_len, B, d_sup, m_sup,
                                                                           mean_entropy);
  return launch_ok();
}

int fopd_refresh_decision(const float *f, const float *m_roll, const float *m_sup, int32_t B, float kappa_f,
                          float kappa_roll, float kappa_sup, int64_t steps_since_refresh, int64_t min_interval,
                          float *means, int32_t *decision, void *stream) {
  if (B <= 0) return FOPD_ERR_SIZE;
  if (!f || !m_roll || !decision) return FOPD_ERR_NULL;
  if (!std::isfinite(kappa_f) || !std::isfinite(kappa_roll) || !std::isfinite(kappa_sup)) return FOPD_ERR_PARAM;
  refresh_decision_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      f, m_roll, m_sup, B, kappa_f, kappa_roll, kappa_sup, steps_since_refresh, min_interval, means, decision);
  return launch_ok();
}

}  // extern "C"
