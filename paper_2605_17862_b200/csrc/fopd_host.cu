// fopd_step_host: the whole batch from host memory.  Only orchestration lives
// here (uploads, the device entry points in order, downloads); every step of
// the path runs in the kernels behind the device entry points.
#include <cuda_runtime.h>

#include <mutex>
#include <vector>

#include "../../include/fopd.h"

namespace {

constexpr uint64_t kAlign = 256;
constexpr uint64_t kPieceBytes = 256ull << 20;  // upload / download granularity of the pipelined path
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


// Uploads the logits of rows [a, b) of a host chunk to the same rows of its device copy, leaving
// out runs of rows with mask = 0: those rows are never read (padding and tool output are a third
// to a half of the batches this path is built for).  Runs of aligned rows separated by a gap
// smaller than 256 KiB go up in one copy.
int upload_logits_rows(const fopd_chunk &c, char *student_dev, char *teacher_dev, int64_t a, int64_t b,
                       cudaStream_t st, uint64_t *h2d_bytes) {
  const uint64_t row_bytes = (uint64_t)c.row_stride * esz(c);
  const int64_t gap = (int64_t)((256u << 10) / row_bytes);
  int64_t n = a;
  while (n < b) {
    while (n < b && c.mask[n] == 0) ++n;
    if (n >= b) break;
    const int64_t lo = n;
    int64_t hi = n + 1;  // one past the last aligned row of the run
    for (int64_t q = hi; q < b && q - hi <= gap; ++q)
      if (c.mask[q] != 0) hi = q + 1;
    CU(cudaMemcpyAsync(student_dev + (uint64_t)lo * row_bytes, static_cast<const char *>(c.student) + (uint64_t)lo * row_bytes,
                       (uint64_t)(hi - lo) * row_bytes, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(teacher_dev + (uint64_t)lo * row_bytes, static_cast<const char *>(c.teacher) + (uint64_t)lo * row_bytes,
                       (uint64_t)(hi - lo) * row_bytes, cudaMemcpyHostToDevice, st));
    *h2d_bytes += 2 * (uint64_t)(hi - lo) * row_bytes;
    n = hi;
  }
  return FOPD_OK;
}

// Streams and events of the pipelined path, one set per device, made on first use and kept.
constexpr int kMaxSlots = 16;
struct Pipe {
  cudaStream_t compute = nullptr, down = nullptr;
  cudaEvent_t up = nullptr, grad = nullptr, fin = nullptr, slot_free[kMaxSlots] = {};
  bool ok = false;
};
std::mutex g_pipe_mu[64];  // one host-buffer step at a time per device: its streams and events are shared state
Pipe g_pipes[64];

int get_pipe(Pipe **out) {
  int d = 0;
  CU(cudaGetDevice(&d));
  if (d < 0 || d >= 64) return FOPD_ERR_CUDA;
  Pipe &P = g_pipes[d];
  if (!P.ok) {
    CU(cudaStreamCreateWithFlags(&P.compute, cudaStreamNonBlocking));
    CU(cudaStreamCreateWithFlags(&P.down, cudaStreamNonBlocking));
    CU(cudaEventCreateWithFlags(&P.up, cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&P.grad, cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&P.fin, cudaEventDisableTiming));
    for (int k = 0; k < kMaxSlots; ++k) CU(cudaEventCreateWithFlags(&P.slot_free[k], cudaEventDisableTiming));
    P.ok = true;
  }
  *out = &P;
  return FOPD_OK;
}

}  // namespace

namespace fopd {
// Destroys the current device's streams and events of the pipelined path (they are made again
// on the next host-buffer step).  Waits for a step in progress on that device.
int host_step_release() {
  int d = 0;
  if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= 64) return FOPD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_pipe_mu[d]);
  Pipe &P = g_pipes[d];
  if (!P.ok) return FOPD_OK;
  bool fine = cudaStreamDestroy(P.compute) == cudaSuccess;
  fine = (cudaStreamDestroy(P.down) == cudaSuccess) && fine;
  fine = (cudaEventDestroy(P.up) == cudaSuccess) && fine;
  fine = (cudaEventDestroy(P.grad) == cudaSuccess) && fine;
  fine = (cudaEventDestroy(P.fin) == cudaSuccess) && fine;
  for (int k = 0; k < kMaxSlots; ++k) fine = (cudaEventDestroy(P.slot_free[k]) == cudaSuccess) && fine;
  P = Pipe();
  if (!fine) (void)cudaGetLastError();
  return fine ? FOPD_OK : FOPD_ERR_CUDA;
}
}  // namespace fopd

namespace {

// rows [a, b) of a chunk as a chunk of its own
fopd_chunk sub_chunk(const fopd_chunk &c, int64_t a, int64_t b) {
  fopd_chunk s = c;
  const int64_t pitch = c.row_stride * esz(c);
  s.student = static_cast<const char *>(c.student) + a * pitch;
  s.teacher = static_cast<const char *>(c.teacher) + a * pitch;
  s.behav_logprob = c.behav_logprob + a;
  s.tokens = c.tokens + a;
  s.mask = c.mask + a;
  s.sample_id = c.sample_id + a;
  s.n_rows = b - a;
  return s;
}

// All logits resident: three streams.  The caller's stream uploads the batch piece by piece;
// the compute stream takes the statistics of each piece as it lands (Algorithm 1's measurement
// phase) and, as soon as every row of a sample has been measured, that sample's freshness and
// the loss and gradient of its rows (the optimisation phase: coef_i depends on sample i alone,
// Eq. 11 and Eq. 16); the download stream returns finished gradient pieces while later rows are
// still arriving, so the two directions of the host link work at the same time.
template <class UploadRows>
int run_pipelined(const fopd_chunk *chunks, const fopd_chunk *dev, int32_t n_chunks, int32_t B, const Layout &L,
                  char *W, float *ws, double *acc, double *lacc, const int32_t *tau_d, const int32_t *len_d,
                  const float *dsup_d, fopd_params p, float *o_f, float *o_w, float *o_dr, float *o_l, float *o_m,
                  float *o_coef, float *o_means, int32_t *status, void *const *dlogits, UploadRows upload_rows,
                  cudaStream_t st, uint64_t *h2d_bytes) {
  int device = 0;
  CU(cudaGetDevice(&device));
  if (device < 0 || device >= 64) return FOPD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_pipe_mu[device]);
  Pipe *P = nullptr;
  RC(get_pipe(&P));
  const uint64_t R = L.rows_total;
  // ready_after[g]: the smallest measured prefix after which row g may be differentiated =
  // one past the last row of any sample met in rows 0..g (prefix maximum of the last occurrences)
  std::vector<uint64_t> last(B, 0), ready_after(R);
  {
    uint64_t g = 0;
    for (int j = 0; j < n_chunks; ++j)
      for (int64_t n = 0; n < chunks[j].n_rows; ++n, ++g) {
        const int32_t s = chunks[j].sample_id[n];
        if (s >= 0 && s < B) last[s] = g + 1;
      }
    uint64_t run = 0;
    g = 0;
    for (int j = 0; j < n_chunks; ++j)
      for (int64_t n = 0; n < chunks[j].n_rows; ++n, ++g) {
        const int32_t s = chunks[j].sample_id[n];
        const uint64_t need = (s >= 0 && s < B) ? last[s] : g + 1;
        run = need > run ? need : run;
        ready_after[g] = run;
      }
  }
  // gradient staging slots
  uint64_t max_row_bytes = 0;
  for (int j = 0; j < n_chunks; ++j) {
    const uint64_t rb = (uint64_t)chunks[j].row_stride * esz(chunks[j]);
    max_row_bytes = rb > max_row_bytes ? rb : max_row_bytes;
  }
  uint64_t slot_bytes = L.logits_bytes_max / 4 < kPieceBytes ? L.logits_bytes_max / 4 : kPieceBytes;
  slot_bytes = up(slot_bytes > max_row_bytes ? slot_bytes : max_row_bytes);
  int n_slots = (int)(up(L.logits_bytes_max) / slot_bytes);
  n_slots = n_slots < 1 ? 1 : (n_slots > kMaxSlots ? kMaxSlots : n_slots);
  bool slot_used[kMaxSlots] = {};
  int next_slot = 0;

  // on any error: let the internal streams drain before the caller may free the workspace
  struct Drain {
    Pipe *P;
    ~Drain() {
      cudaStreamSynchronize(P->compute);
      cudaStreamSynchronize(P->down);
    }
  } drain{P};

  CU(cudaEventRecord(P->up, st));
  CU(cudaStreamWaitEvent(P->compute, P->up, 0));
  uint64_t measured = 0, graded = 0;  // global row counts
  int gj = 0;                          // chunk the next row to differentiate lies in
  auto differentiate = [&](uint64_t upto) -> int {
    RC(fopd_sample_freshness(acc, tau_d, len_d, dsup_d, B, p, o_f, o_w, o_dr, o_l, o_m, o_coef, o_means, status,
                             P->compute));
    while (graded < upto) {
      while (gj < n_chunks && graded >= L.row_off[gj] + (uint64_t)chunks[gj].n_rows) ++gj;
      const fopd_chunk &c = chunks[gj];
      const uint64_t row_bytes = (uint64_t)c.row_stride * esz(c);
      const int64_t a = (int64_t)(graded - L.row_off[gj]);
      int64_t b = (int64_t)((upto < L.row_off[gj] + (uint64_t)c.n_rows ? upto : L.row_off[gj] + (uint64_t)c.n_rows) -
                            L.row_off[gj]);
      const int64_t cap = (int64_t)(slot_bytes / row_bytes);
      if (b - a > cap) b = a + cap;
      const int k = next_slot;
      next_slot = (next_slot + 1) % n_slots;
      void *slot = W + L.ds_off + (uint64_t)k * slot_bytes;
      if (slot_used[k]) CU(cudaStreamWaitEvent(P->compute, P->slot_free[k], 0));
      const fopd_chunk piece = sub_chunk(dev[gj], a, b);
      RC(fopd_loss_fwd_bwd(&piece, B, o_coef, ws + 4 * (L.row_off[gj] + (uint64_t)a), p, slot, lacc, status,
                           P->compute));
      CU(cudaEventRecord(P->grad, P->compute));
      CU(cudaStreamWaitEvent(P->down, P->grad, 0));
      CU(cudaMemcpyAsync(static_cast<char *>(dlogits[gj]) + (uint64_t)a * row_bytes, slot,
                         (uint64_t)(b - a) * row_bytes, cudaMemcpyDeviceToHost, P->down));
      CU(cudaEventRecord(P->slot_free[k], P->down));
      slot_used[k] = true;
      graded += (uint64_t)(b - a);
    }
    return FOPD_OK;
  };
  for (int j = 0; j < n_chunks; ++j) {
    const fopd_chunk &c = chunks[j];
    if (c.n_rows == 0) continue;
    RC(upload_rows(j));
    const uint64_t row_bytes = (uint64_t)c.row_stride * esz(c);
    const int64_t step = (int64_t)(slot_bytes / row_bytes);
    for (int64_t a = 0; a < c.n_rows; a += step) {
      const int64_t b = a + step < c.n_rows ? a + step : c.n_rows;
      RC(upload_logits_rows(c, W + L.s_off[j], W + L.t_off[j], a, b, st, h2d_bytes));
      CU(cudaEventRecord(P->up, st));
      CU(cudaStreamWaitEvent(P->compute, P->up, 0));
      const fopd_chunk piece = sub_chunk(dev[j], a, b);
      RC(fopd_token_stats(&piece, B, nullptr, nullptr, nullptr, nullptr, ws + 4 * (L.row_off[j] + (uint64_t)a), acc,
                          status, P->compute));
      measured = L.row_off[j] + (uint64_t)b;
      // rows whose samples are complete within the measured prefix
      uint64_t upto = graded;
      while (upto < R && ready_after[upto] <= measured) ++upto;
      if (upto > graded) RC(differentiate(upto));
    }
  }
  // outputs of every sample from the complete sums (again: samples without rows, empty batches)
  RC(fopd_sample_freshness(acc, tau_d, len_d, dsup_d, B, p, o_f, o_w, o_dr, o_l, o_m, o_coef, o_means, status,
                           P->compute));
  if (graded != R) return FOPD_ERR_SIZE;
  CU(cudaEventRecord(P->fin, P->compute));
  CU(cudaStreamWaitEvent(st, P->fin, 0));
  CU(cudaEventRecord(P->grad, P->down));
  CU(cudaStreamWaitEvent(st, P->grad, 0));
  return FOPD_OK;
}

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

  uint64_t h2d_bytes = (uint64_t)B * (d_sup ? 12 : 8), d2h_bytes = sizeof(int32_t);
  std::vector<fopd_chunk> dev(n_chunks);
  auto upload_logits = [&](int j) -> int {
    return upload_logits_rows(chunks[j], W + L.s_off[j], W + L.t_off[j], 0, chunks[j].n_rows, st, &h2d_bytes);
  };
  for (int j = 0; j < n_chunks; ++j) {
    const uint64_t r0 = L.row_off[j];
    dev[j] = chunks[j];
    dev[j].student = at(L.s_off[j]);
    dev[j].teacher = at(L.t_off[j]);
    dev[j].behav_logprob = behav + r0;
    dev[j].tokens = tok + r0;
    dev[j].mask = mask + r0;
    dev[j].sample_id = sid + r0;
    if (chunks[j].n_rows > 0 && !dlogits[j]) return FOPD_ERR_NULL;
  }
  auto upload_rows = [&](int j) -> int {
    const fopd_chunk &c = chunks[j];
    const uint64_t r0 = L.row_off[j];
    const size_t n = (size_t)c.n_rows;
    CU(cudaMemcpyAsync(behav + r0, c.behav_logprob, n * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(tok + r0, c.tokens, n * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(sid + r0, c.sample_id, n * 4, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(mask + r0, c.mask, n, cudaMemcpyHostToDevice, st));
    h2d_bytes += 13 * (uint64_t)n;
    d2h_bytes += (uint64_t)n * c.row_stride * esz(c);  // the chunk's gradient, returned in either mode
    return FOPD_OK;
  };
  if (resident) {
    RC(run_pipelined(chunks, dev.data(), n_chunks, B, L, W, ws, acc, lacc, tau_d, len_d, dsup_d, p, o_f, o_w, o_dr,
                     o_l, o_m, o_coef, o_means, status, dlogits, upload_rows, st, &h2d_bytes));
  } else {
    // Measurement phase (Algorithm 1, first loop): statistics of every chunk.
    for (int j = 0; j < n_chunks; ++j) {
      if (chunks[j].n_rows == 0) continue;
      RC(upload_logits(j));
      RC(upload_rows(j));
      RC(fopd_token_stats(&dev[j], B, nullptr, nullptr, nullptr, nullptr, ws + 4 * L.row_off[j], acc, status, st));
    }
    RC(fopd_sample_freshness(acc, tau_d, len_d, dsup_d, B, p, o_f, o_w, o_dr, o_l, o_m, o_coef, o_means, status,
                             st));
    // Optimisation phase (Algorithm 1, minibatch loop): loss and gradient.
    for (int j = 0; j < n_chunks; ++j) {
      const size_t n = (size_t)chunks[j].n_rows;
      if (n == 0) continue;
      RC(upload_logits(j));
      RC(fopd_loss_fwd_bwd(&dev[j], B, o_coef, ws + 4 * L.row_off[j], p, at(L.ds_off), lacc, status, st));
      CU(cudaMemcpyAsync(dlogits[j], at(L.ds_off), n * chunks[j].row_stride * esz(chunks[j]),
                         cudaMemcpyDeviceToHost, st));
    }
  }
  RC(fopd_loss_finalize(lacc, acc, o_w, B, p, o_per, o_loss, st));
  auto down = [&](float *dst, const float *src, size_t n) -> int {
    if (dst) {
      CU(cudaMemcpyAsync(dst, src, n * 4, cudaMemcpyDeviceToHost, st));
      d2h_bytes += n * 4;
    }
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
  if (out->copied_bytes) {
    out->copied_bytes[0] = (int64_t)h2d_bytes;
    out->copied_bytes[1] = (int64_t)d2h_bytes;
  }
  return bits == 0 ? FOPD_OK : FOPD_ERR_DEVICE;
}

}  // extern "C"
