// fopd_step_host: the whole batch from host memory.  Only orchestration lives
// here (uploads, the device entry points in order, downloads); every step of
// the path runs in the kernels behind the device entry points.
#include <cuda_runtime.h>

#include <vector>

#include "../../include/fopd.h"

namespace {

constexpr uint64_t kAlign = 256;
uint64_t up(uint64_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  uint64_t total = 0;
  uint64_t logits_bytes_max = 0;  // largest chunk, one tensor
  uint64_t rows_total = 0;
  std::vector<uint64_t> s_off, t_off, row_off;  // per chunk
  uint64_t ds_off = 0, behav_off = 0, tok_off = 0, mask_off = 0, sid_off = 0, ws_off = 0;
  uint64_t acc_off = 0, lacc_off = 0, tau_off = 0, len_off = 0, dsup_off = 0, outs_off = 0, status_off = 0;
};

int esz(const fopd_chunk &c) { return c.dtype == FOPD_BF16 ? 2 : 4; }

Layout make_layout(const fopd_chunk *chunks, int32_t n_chunks, int32_t B, bool resident) {
  Layout L;
  uint64_t off = 0;
  L.s_off.resize(n_chunks);
  L.t_off.resize(n_chunks);
  L.row_off.resize(n_chunks);
  for (int j = 0; j < n_chunks; ++j) {
    const uint64_t bytes = (uint64_t)chunks[j].n_rows * chunks[j].row_stride * esz(chunks[j]);
    if (bytes > L.logits_bytes_max) L.logits_bytes_max = bytes;
    L.row_off[j] = L.rows_total;
    L.rows_total += (uint64_t)chunks[j].n_rows;
  }
  if (resident) {
    for (int j = 0; j < n_chunks; ++j) {
      const uint64_t bytes = up((uint64_t)chunks[j].n_rows * chunks[j].row_stride * esz(chunks[j]));
      L.s_off[j] = off;
      off += bytes;
      L.t_off[j] = off;
      off += bytes;
    }
  } else {
    for (int j = 0; j < n_chunks; ++j) {
      L.s_off[j] = off;
      L.t_off[j] = off + up(L.logits_bytes_max);
    }
    off += 2 * up(L.logits_bytes_max);
  }
  L.ds_off = off;
  off += up(L.logits_bytes_max);
  const uint64_t R = L.rows_total;
  L.behav_off = off; off += up(R * 4);
  L.tok_off = off;   off += up(R * 4);
  L.sid_off = off;   off += up(R * 4);
  L.mask_off = off;  off += up(R);
  L.ws_off = off;    off += up(R * 16);
  L.acc_off = off;   off += up((uint64_t)B * 32);
  L.lacc_off = off;  off += up((uint64_t)B * 16);
  L.tau_off = off;   off += up((uint64_t)B * 4);
  L.len_off = off;   off += up((uint64_t)B * 4);
  L.dsup_off = off;  off += up((uint64_t)B * 4);
  L.outs_off = off;  off += up((uint64_t)B * 4) * 7 + up(16);  // f w d_roll l m coef per_sample | means, loss
  L.status_off = off; off += kAlign;
  L.total = off;
  return L;
}

int check_host_chunks(const fopd_chunk *chunks, int32_t n_chunks, int32_t B) {
  if (!chunks) return FOPD_ERR_NULL;
  if (n_chunks <= 0 || B <= 0) return FOPD_ERR_SIZE;
  for (int j = 0; j < n_chunks; ++j) {
    const fopd_chunk &c = chunks[j];
    if (c.dtype != FOPD_BF16 && c.dtype != FOPD_F32) return FOPD_ERR_DTYPE;
    if (c.n_rows < 0 || c.vocab <= 0 || c.row_stride < c.vocab) return FOPD_ERR_SIZE;
    if ((c.row_stride * esz(c)) % 16 != 0) return FOPD_ERR_ALIGN;
    if (c.n_rows > 0 && (!c.student || !c.teacher || !c.behav_logprob || !c.tokens || !c.mask || !c.sample_id))
      return FOPD_ERR_NULL;
  }
  return FOPD_OK;
}

#define CU(x)                                  \
  do {                                         \
    if ((x) != cudaSuccess) return FOPD_ERR_CUDA; \
  } while (0)
#define RC(x)                     \
  do {                            \
    int rc_ = (x);                \
    if (rc_ != FOPD_OK) return rc_; \
  } while (0)

}  // namespace

extern "C" {

uint64_t fopd_step_host_workspace_bytes(const fopd_chunk *chunks, int32_t n_chunks, int32_t B,
                                        int32_t resident) {
  if (check_host_chunks(chunks, n_chunks, B) != FOPD_OK) return 0;
  return make_layout(chunks, n_chunks, B, resident != 0).total;
}

int fopd_step_host(const fopd_chunk *chunks, int32_t n_chunks, int32_t B, const int32_t *staleness,
                   const int32_t *seq_len, const float *d_sup, fopd_params p, void *const *dlogits,
                   const fopd_host_outputs *out, void *workspace, uint64_t workspace_bytes, void *stream) {
  RC(check_host_chunks(chunks, n_chunks, B));
  if (!staleness || !seq_len || !dlogits || !out || !out->loss || !workspace) return FOPD_ERR_NULL;
  if (((uintptr_t)workspace & (kAlign - 1)) != 0) return FOPD_ERR_ALIGN;
  bool resident = true;
  Layout L = make_layout(chunks, n_chunks, B, true);
  if (L.total > workspace_bytes) {
    resident = false;
    L = make_layout(chunks, n_chunks, B, false);
    if (L.total > workspace_bytes) return FOPD_ERR_SIZE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char *W = static_cast<char *>(workspace);
  auto at = [&](uint64_t off) { return static_cast<void *>(W + off); };
  float *behav = static_cast<float *>(at(L.behav_off));
  int32_t *tok = static_cast<int32_t *>(at(L.tok_off));
  int32_t *sid = static_cast<int32_t *>(at(L.sid_off));
  uint8_t *mask = static_cast<uint8_t *>(at(L.mask_off));
  float *ws = static_cast<float *>(at(L.ws_off));
  double *acc = static_cast<double *>(at(L.acc_off));
  double *lacc = static_cast<double *>(at(L.lacc_off));
  int32_t *tau_d = static_cast<int32_t *>(at(L.tau_off));
  int32_t *len_d = static_cast<int32_t *>(at(L.len_off));
  float *dsup_d = d_sup ? static_cast<float *>(at(L.dsup_off)) : nullptr;
  const uint64_t ob = up((uint64_t)B * 4);
  float *o_f = static_cast<float *>(at(L.outs_off)), *o_w = static_cast<float *>(at(L.outs_off + ob));
  float *o_dr = static_cast<float *>(at(L.outs_off + 2 * ob)), *o_l = static_cast<float *>(at(L.outs_off + 3 * ob));
  float *o_m = static_cast<float *>(at(L.outs_off + 4 * ob)), *o_coef = static_cast<float *>(at(L.outs_off + 5 * ob));
  float *o_per = static_cast<float *>(at(L.outs_off + 6 * ob));
  float *o_means = static_cast<float *>(at(L.outs_off + 7 * ob)), *o_loss = o_means + 2;
  int32_t *status = static_cast<int32_t *>(at(L.status_off));

  CU(cudaMemsetAsync(acc, 0, (size_t)B * 32, st));
  CU(cudaMemsetAsync(lacc, 0, (size_t)B * 16, st));
  CU(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
  CU(cudaMemcpyAsync(tau_d, staleness, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(len_d, seq_len, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  if (d_sup) CU(cudaMemcpyAsync(dsup_d, d_sup, (size_t)B * 4, cudaMemcpyHostToDevice, st));

  std::vector<fopd_chunk> dev(n_chunks);
  auto upload_logits = [&](int j) -> int {
    const size_t bytes = (size_t)chunks[j].n_rows * chunks[j].row_stride * esz(chunks[j]);
    if (bytes == 0) return FOPD_OK;
    CU(cudaMemcpyAsync(at(L.s_off[j]), chunks[j].student, bytes, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(at(L.t_off[j]), chunks[j].teacher, bytes, cudaMemcpyHostToDevice, st));
    return FOPD_OK;
  };
  // Measurement phase (Algorithm 1, first loop): statistics of every chunk.
  for (int j = 0; j < n_chunks; ++j) {
    const fopd_chunk &c = chunks[j];
    const uint64_t r0 = L.row_off[j];
    const size_t n = (size_t)c.n_rows;
    dev[j] = c;
    dev[j].student = at(L.s_off[j]);
    dev[j].teacher = at(L.t_off[j]);
    dev[j].behav_logprob = behav + r0;
    dev[j].tokens = tok + r0;
    dev[j].mask = mask + r0;
    dev[j].sample_id = sid + r0;
    if (n == 0) continue;
    RC(upload_logits(j));
    CU(cudaMemcpyAsync(behav + r0, c.behav_logprob, n * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(tok + r0, c.tokens, n * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(sid + r0, c.sample_id, n * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(mask + r0, c.mask, n, cudaMemcpyHostToDevice, st));
    RC(fopd_token_stats(&dev[j], B, nullptr, nullptr, nullptr, nullptr, ws + 4 * r0, acc, status, st));
  }
  RC(fopd_sample_freshness(acc, tau_d, len_d, dsup_d, B, p, o_f, o_w, o_dr, o_l, o_m, o_coef, o_means, status, st));
  // Optimisation phase (Algorithm 1, minibatch loop): loss and gradient.
  for (int j = 0; j < n_chunks; ++j) {
    const size_t n = (size_t)chunks[j].n_rows;
    if (n == 0) continue;
    if (!dlogits[j]) return FOPD_ERR_NULL;
    if (!resident) RC(upload_logits(j));
    RC(fopd_loss_fwd_bwd(&dev[j], B, o_coef, ws + 4 * L.row_off[j], p, at(L.ds_off), lacc, status, st));
    CU(cudaMemcpyAsync(dlogits[j], at(L.ds_off), n * chunks[j].row_stride * esz(chunks[j]),
                       cudaMemcpyDeviceToHost, st));
  }
  RC(fopd_loss_finalize(lacc, acc, o_w, B, p, o_per, o_loss, st));
  auto down = [&](float *dst, const float *src, size_t n) -> int {
    if (dst) CU(cudaMemcpyAsync(dst, src, n * 4, cudaMemcpyDeviceToHost, st));
    return FOPD_OK;
  };
  RC(down(out->f, o_f, B));
  RC(down(out->w, o_w, B));
  RC(down(out->d_roll, o_dr, B));
  RC(down(out->l_distill, o_l, B));
  RC(down(out->m_align, o_m, B));
  RC(down(out->per_sample_loss, o_per, B));
  RC(down(out->buffer_means, o_means, 2));
  RC(down(out->loss, o_loss, 1));
  int32_t bits = 0;
  CU(cudaMemcpyAsync(&bits, status, sizeof(bits), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  if (out->status_bits) *out->status_bits = bits;
  return bits == 0 ? FOPD_OK : FOPD_ERR_DEVICE;
}

}  // extern "C"
