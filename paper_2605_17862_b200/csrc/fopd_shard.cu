// Entry points for vocabulary-sharded rows: partial sums of one shard, merge of
// all parts into the row statistics, gradient of one shard's columns.
#include "host_common.cuh"
#include "shard_kernels.cuh"

using namespace fopd;

namespace {

int check_shard(const fopd_chunk *shard, int64_t vocab_offset, int64_t vocab_total) {
  int rc = check_chunk(shard, 1);
  if (rc != FOPD_OK) return rc;
  if (shard->loss_kind != FOPD_LOSS_FULL_KL) return FOPD_ERR_KIND;
  if (vocab_offset < 0 || vocab_total > (int64_t)1 << 30 || vocab_offset + shard->vocab > vocab_total)
    return FOPD_ERR_SIZE;
  return FOPD_OK;
}

// The per-row side arrays of a chunk without its logits, judged against the full vocabulary.
int check_rows(const fopd_chunk *rows, int32_t B) {
  if (!rows) return FOPD_ERR_NULL;
  if (rows->loss_kind != FOPD_LOSS_FULL_KL) return FOPD_ERR_KIND;
  if (rows->n_rows < 0 || rows->vocab <= 0 || rows->vocab > (int64_t)1 << 30 || B <= 0) return FOPD_ERR_SIZE;
  if (rows->n_rows > 0 && (!rows->behav_logprob || !rows->tokens || !rows->mask || !rows->sample_id))
    return FOPD_ERR_NULL;
  return FOPD_OK;
}

}  // namespace

extern "C" {

int fopd_shard_stats(const fopd_chunk *shard, int64_t vocab_offset, int64_t vocab_total, float *partial,
                     void *stream) {
  int rc = check_shard(shard, vocab_offset, vocab_total);
  if (rc != FOPD_OK) return rc;
  if (shard->n_rows == 0) return FOPD_OK;
  if (!partial) return FOPD_ERR_NULL;
  if (!aligned16(partial)) return FOPD_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ChunkDev d = to_dev(shard);
  const unsigned grid = row_grid(shard->n_rows);
  const bool short_row = shard->vocab / (shard->dtype == FOPD_BF16 ? 8 : 4) < kShortRowVecs;
#define FOPD_LAUNCH(DT, T) shard_stats_kernel<DT, T><<<grid, T, 0, st>>>(d, vocab_offset, partial)
  if (shard->dtype == FOPD_BF16) {
    if (short_row) FOPD_LAUNCH(FOPD_BF16, kStatsThreadsShortRow);
    else FOPD_LAUNCH(FOPD_BF16, kStatsThreads);
  } else {
    if (short_row) FOPD_LAUNCH(FOPD_F32, kStatsThreadsShortRow);
    else FOPD_LAUNCH(FOPD_F32, kStatsThreads);
  }
#undef FOPD_LAUNCH
  return launch_ok();
}

int fopd_shard_merge(const float *partials, int32_t n_parts, const fopd_chunk *rows, int32_t B, float *lp_s,
                     float *lp_t, float *kl, float *ratio, float *row_ws, double *acc, int32_t *status,
                     void *stream) {
  int rc = check_rows(rows, B);
  if (rc != FOPD_OK) return rc;
  if (n_parts <= 0) return FOPD_ERR_SIZE;
  if (!acc) return FOPD_ERR_NULL;
  if (rows->n_rows == 0) return FOPD_OK;
  if (!partials || !row_ws) return FOPD_ERR_NULL;
  if (!aligned16(partials) || !aligned16(row_ws)) return FOPD_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ChunkDev d = to_dev(rows);
  shard_merge_kernel<<<(unsigned)((rows->n_rows + 255) / 256), 256, 0, st>>>(partials, n_parts, d, B, lp_s, lp_t, kl,
                                                                           ratio, row_ws, status);
  if ((rc = launch_ok()) != FOPD_OK) return rc;
  return launch_segment_reduce(d, B, row_ws, nullptr, 0, acc, st);
}

int fopd_shard_loss_fwd_bwd(const fopd_chunk *shard, int64_t vocab_offset, int64_t vocab_total, int32_t B,
                            const float *coef, const float *row_ws, fopd_params p, void *dlogits, double *loss_acc,
                            void *stream) {
  int rc = check_shard(shard, vocab_offset, vocab_total);
  if (rc != FOPD_OK) return rc;
  if (B <= 0) return FOPD_ERR_SIZE;
  if ((rc = check_params(p)) != FOPD_OK) return rc;
  if (!coef) return FOPD_ERR_NULL;
  if (shard->n_rows == 0) return FOPD_OK;
  if (!dlogits || !row_ws) return FOPD_ERR_NULL;
  if (!aligned16(dlogits) || !aligned16(row_ws)) return FOPD_ERR_ALIGN;
  {
    // extents of the three views, from the first column of the first row to the last of the last
    const int64_t esz = shard->dtype == FOPD_BF16 ? 2 : 4;
    const uintptr_t bytes = (uintptr_t)(((shard->n_rows - 1) * shard->row_stride + shard->vocab) * esz);
    const uintptr_t o = (uintptr_t)dlogits, s = (uintptr_t)shard->student, t = (uintptr_t)shard->teacher;
    if ((o < s + bytes && s < o + bytes) || (o < t + bytes && t < o + bytes)) return FOPD_ERR_ALIAS;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ChunkDev d = to_dev(shard);
  const unsigned grid = row_grid(shard->n_rows);
  const bool short_row = shard->vocab / (shard->dtype == FOPD_BF16 ? 8 : 4) < kShortRowVecs;
#define FOPD_LAUNCH(DT, T) \
  shard_grad_kernel<DT, T><<<grid, T, 0, st>>>(d, vocab_offset, vocab_total, B, coef, row_ws, p.lambda, dlogits)
  if (shard->dtype == FOPD_BF16) {
    if (short_row) FOPD_LAUNCH(FOPD_BF16, kGradThreadsShortRow);
    else FOPD_LAUNCH(FOPD_BF16, kGradThreads);
  } else {
    if (short_row) FOPD_LAUNCH(FOPD_F32, kGradThreadsShortRow);
    else FOPD_LAUNCH(FOPD_F32, kGradThreads);
  }
#undef FOPD_LAUNCH
  if ((rc = launch_ok()) != FOPD_OK) return rc;
  if (loss_acc) {  // the sums do not depend on the shard: every holder gets the same, or one holder asks
    ChunkDev whole = d;
    whole.vocab = vocab_total;
    rc = launch_segment_reduce(whole, B, row_ws, coef, 1, loss_acc, st);
  }
  return rc;
}

}  // extern "C"
