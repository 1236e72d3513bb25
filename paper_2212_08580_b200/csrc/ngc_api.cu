// C-ABI entry points that touch the GPU: argument checks, lazily created device tables and
// workspace, and the launch sequences of the hot path.
#include <cstdio>
#include <cstring>
#include <vector>

#include "ngc_device.h"

namespace ngc {
int device_sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}
}  // namespace ngc

namespace {

#define NGC_CUDA(p, call)                      \
  do {                                         \
    cudaError_t e__ = (call);                  \
    if (e__ != cudaSuccess) {                  \
      (p)->last_cuda = (int)e__;               \
      return NGC_ERR_CUDA;                     \
    }                                          \
  } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int ensure_tables(ngc_plan_s *p) {
  if (p->tables_on_device) return NGC_OK;
  int dev = 0;
  NGC_CUDA(p, cudaGetDevice(&dev));
  p->device = dev;
  for (auto &lv : p->lv) {
    NGC_CUDA(p, cudaMalloc(&lv.d_coef, lv.coef.size() * sizeof(double)));
    NGC_CUDA(p, cudaMemcpy(lv.d_coef, lv.coef.data(), lv.coef.size() * sizeof(double), cudaMemcpyHostToDevice));
    NGC_CUDA(p, cudaMalloc(&lv.d_a0, lv.a0.size() * sizeof(double)));
    NGC_CUDA(p, cudaMemcpy(lv.d_a0, lv.a0.data(), lv.a0.size() * sizeof(double), cudaMemcpyHostToDevice));
    if (!lv.N.empty()) {
      NGC_CUDA(p, cudaMalloc(&lv.d_N, lv.N.size() * sizeof(double)));
      NGC_CUDA(p, cudaMemcpy(lv.d_N, lv.N.data(), lv.N.size() * sizeof(double), cudaMemcpyHostToDevice));
    }
  }
  NGC_CUDA(p, cudaMalloc(&p->d_status, 2 * sizeof(int)));
  NGC_CUDA(p, cudaMemset(p->d_status, 0, 2 * sizeof(int)));
  NGC_CUDA(p, cudaMalloc(&p->d_maxres, sizeof(double)));
  NGC_CUDA(p, cudaMemset(p->d_maxres, 0, sizeof(double)));
  p->tables_on_device = true;
  return NGC_OK;
}

int ensure_ws(ngc_plan_s *p, size_t bytes) {
  if (bytes <= p->ws_bytes) return NGC_OK;
  if (p->ws) {
    NGC_CUDA(p, cudaDeviceSynchronize());
    NGC_CUDA(p, cudaFree(p->ws));
    p->ws = nullptr;
    p->ws_bytes = 0;
  }
  NGC_CUDA(p, cudaMalloc(&p->ws, bytes));
  p->ws_bytes = bytes;
  return NGC_OK;
}

int ensure_batch(ngc_plan_s *p, int batch) {
  if (batch <= p->a_batch_cap) return NGC_OK;
  if (p->d_a) {
    NGC_CUDA(p, cudaDeviceSynchronize());
    cudaFree(p->d_a);
    cudaFree(p->d_resid);
    cudaFree(p->d_masks);
    p->d_a = nullptr; p->d_resid = nullptr; p->d_masks = nullptr; p->a_batch_cap = 0;
  }
  NGC_CUDA(p, cudaMalloc(&p->d_a, (size_t)batch * p->n * sizeof(double)));
  NGC_CUDA(p, cudaMalloc(&p->d_resid, (size_t)batch * sizeof(double)));
  NGC_CUDA(p, cudaMalloc(&p->d_masks, (size_t)batch * 2 * sizeof(uint64_t)));
  p->a_batch_cap = batch;
  return NGC_OK;
}

int ensure_staging(ngc_plan_s *p, void **buf, size_t *have, size_t want) {
  if (want <= *have) return NGC_OK;
  if (*buf) {
    NGC_CUDA(p, cudaDeviceSynchronize());
    NGC_CUDA(p, cudaFree(*buf));
    *buf = nullptr;
    *have = 0;
  }
  NGC_CUDA(p, cudaMalloc(buf, want));
  *have = want;
  return NGC_OK;
}

// Checks a responsive set and packs it into a bit mask.
int pack_set(const ngc_plan_s *p, int layer, const int32_t *S, int nS, uint64_t *mask) {
  const int n = p->n, s = p->lv[layer].s;
  if (!S || nS < n - s || nS > n) return NGC_ERR_INVALID;
  mask[0] = mask[1] = 0;
  for (int t = 0; t < nS; ++t) {
    if (S[t] < 0 || S[t] >= n) return NGC_ERR_INVALID;
    if (t > 0 && S[t] <= S[t - 1]) return NGC_ERR_INVALID;
    mask[S[t] >> 6] |= 1ull << (S[t] & 63);
  }
  return NGC_OK;
}

int check_model(const ngc_plan_s *p, const ngc_model_t *m) {
  if (!m || m->rows_per_partition < 1 || m->d < 1) return NGC_ERR_INVALID;
  if (ngc_num_params(m) < 0) return NGC_ERR_INVALID;
  if (m->x_dtype != NGC_F32 && m->x_dtype != NGC_BF16) return NGC_ERR_INVALID;
  (void)p;
  return NGC_OK;
}

// Records one event of a begin/end pair on `stream` when profiling is on.
int profile_mark(ngc_plan_s *p, cudaStream_t stream) {
  if (!p->profiling) return NGC_OK;
  if (p->ev_used == p->ev.size()) {
    cudaEvent_t e;
    NGC_CUDA(p, cudaEventCreate(&e));
    p->ev.push_back(e);
  }
  NGC_CUDA(p, cudaEventRecord(static_cast<cudaEvent_t>(p->ev[p->ev_used++]), stream));
  return NGC_OK;
}

// The residual |a B - 1| above which a decode is reported as NGC_ERR_SINGULAR.
constexpr double kResidualLimit = 1e-6;

}  // namespace

extern "C" {

void ngc_plan_destroy(ngc_plan_t *p) {
  if (!p) return;
  if (p->tables_on_device || p->ws || p->st_X || p->dense_state) {
    cudaDeviceSynchronize();
    for (auto &lv : p->lv) {
      cudaFree(lv.d_coef);
      cudaFree(lv.d_a0);
      cudaFree(lv.d_N);
    }
    cudaFree(p->ws);
    cudaFree(p->d_a);
    cudaFree(p->d_resid);
    cudaFree(p->d_masks);
    cudaFree(p->d_status);
    cudaFree(p->d_maxres);
    cudaFree(p->d_gpart);
    cudaFree(p->d_shard_coef);
    cudaFree(p->d_shard_a);
    cudaFree(p->st_X);
    cudaFree(p->st_y);
    cudaFree(p->st_theta);
    cudaFree(p->st_coded);
    cudaFree(p->st_grad);
  }
  ngc::dense_state_free(static_cast<ngc::DenseState *>(p->dense_state));
  for (void *e : p->ev) cudaEventDestroy(static_cast<cudaEvent_t>(e));
  if (p->ev_solved) cudaEventDestroy(static_cast<cudaEvent_t>(p->ev_solved));
  if (p->ev_decoded) cudaEventDestroy(static_cast<cudaEvent_t>(p->ev_decoded));
  if (p->ev_grads) cudaEventDestroy(static_cast<cudaEvent_t>(p->ev_grads));
  if (p->side_stream) cudaStreamDestroy(static_cast<cudaStream_t>(p->side_stream));
  delete p;
}

}  // extern "C"

namespace {

// What ngc_step hands to the gradient + encode launcher so that the decode can ride on the encode kernel
// of the dense models: the event after which the decoding vector is on the device, where the decoded
// gradient goes, and whether the encode took the decode along.
struct DecodeHook {
  cudaEvent_t solved;
  float *grad;
  bool fused;
  cudaEvent_t after_grads;  // if set: recorded on the caller's stream right behind the gradient kernels
};

int grad_encode_impl(ngc_plan_t *p, const ngc_model_t *m, const void *theta, const void *X, const void *y, int layer,
                     void *coded, void *cuda_stream, DecodeHook *hook);

}  // namespace

extern "C" {

int ngc_grad_encode(ngc_plan_t *p, const ngc_model_t *m, const void *theta, const void *X, const void *y, int layer,
                    void *coded, void *cuda_stream) {
  return grad_encode_impl(p, m, theta, X, y, layer, coded, cuda_stream, nullptr);
}

}  // extern "C"

namespace {

// Encode of a dense model's partial gradients; with a hook, the decode in the same kernel.
int encode_dense(ngc_plan_t *p, const ngc::RowSplit &split, const float *G, long long ldG, const ngc_level_t &lv,
                 long long l, void *coded, int cdt, cudaStream_t stream, DecodeHook *hook) {
  if (!hook || !hook->grad) {  // no decode to take along (or its vector is not solved before the encode)
    NGC_CUDA(p, ngc::launch_encode_long(split, G, ldG, lv.d_coef, p->n, lv.s, l, coded, cdt, stream));
    return NGC_OK;
  }
  const int rc = ensure_staging(p, &p->d_gpart, &p->gpart_bytes, (size_t)ngc::kEncodeMaxChunks * l * sizeof(double));
  if (rc != NGC_OK) return rc;
  NGC_CUDA(p, cudaStreamWaitEvent(stream, hook->solved, 0));
  int sum_launches = 0;
  ngc::EncodeDecodeArgs dec{p->d_a, static_cast<double *>(p->d_gpart), hook->grad, &hook->fused, &sum_launches};
  NGC_CUDA(p, ngc::launch_encode_long(split, G, ldG, lv.d_coef, p->n, lv.s, l, coded, cdt, stream, &dec));
  p->launches += sum_launches;  // the sum over the worker chunks, when there are several
  return NGC_OK;
}

// Where the gradient kernels left the partial gradients of the partition groups: fp32 [group][slot][ld], the
// slots of a group to be added up in order (see RowSplit).
struct PartialGrads {
  ngc::RowSplit split;
  const float *ws;
  long long ld;
  int launches;
};

// Partial gradients g_j of `n_groups` consecutive partition groups (q partitions each) whose data start at X / y:
// the gradient kernels of the model kind, into the plan's scratch.  The whole problem is n_groups = n; a shard of
// it passes fewer.
int partial_gradients(ngc_plan_t *p, const ngc_model_t *m, const void *theta, const void *X, const void *y, int n_groups,
                      cudaStream_t stream, PartialGrads *out) {
  int rc;
  const int sms = ngc::device_sm_count();
  if (sms <= 0) { p->last_cuda = (int)cudaErrorNoDevice; return NGC_ERR_CUDA; }
  const int k = n_groups * p->q;
  if (m->kind == NGC_LSQ || m->kind == NGC_LOGISTIC) {
    const int vec = (m->x_dtype == NGC_F32) ? 4 : 8;
    if (m->d % vec != 0 || m->d / vec > 4 * 512) return NGC_ERR_INVALID;  // rows must be whole 16-byte vectors
    out->split = ngc::make_row_split(n_groups, (long long)p->q * m->rows_per_partition, sms);
    rc = ensure_ws(p, (size_t)n_groups * out->split.P * m->d * sizeof(float));
    if (rc != NGC_OK) return rc;
    if ((rc = profile_mark(p, stream)) != NGC_OK) return rc;
    NGC_CUDA(p, ngc::launch_gemv_pair(*m, out->split, X, static_cast<const float *>(y), static_cast<const float *>(theta),
                                      static_cast<float *>(p->ws), p->d_status, stream));
    if ((rc = profile_mark(p, stream)) != NGC_OK) return rc;
    out->ws = static_cast<const float *>(p->ws);
    out->ld = m->d;
    out->launches = 1;
    return NGC_OK;
  }
  // dense models: one scratch slot per partition, a group is q consecutive partitions
  out->split.T = k; out->split.rows_g = p->q; out->split.grid = k; out->split.P = p->q;
  float *G = nullptr;
  if (m->kind == NGC_SOFTMAX) {
    if (m->x_dtype != NGC_BF16 || m->n_classes % 16 != 0 || m->n_classes < 16 || m->n_classes > 256 || m->d % 8 != 0)
      return NGC_ERR_INVALID;
    rc = ensure_ws(p, ngc::softmax_scratch_bytes(k, m->rows_per_partition, m->d, m->n_classes));
    if (rc != NGC_OK) return rc;
    if ((rc = profile_mark(p, stream)) != NGC_OK) return rc;
    NGC_CUDA(p, ngc::launch_softmax_grad(k, m->rows_per_partition, m->d, m->n_classes, X, static_cast<const int *>(y),
                                         static_cast<const float *>(theta), static_cast<unsigned char *>(p->ws), &G,
                                         p->d_status, sms, stream,
                                         reinterpret_cast<ngc::DenseState **>(&p->dense_state)));
    if ((rc = profile_mark(p, stream)) != NGC_OK) return rc;
    out->ws = G;
    out->ld = ngc_num_params(m);
    out->launches = 3;
    return NGC_OK;
  }
  if (m->kind == NGC_MLP) {
    if (m->x_dtype != NGC_F32) return NGC_ERR_INVALID;
    const int h = m->hidden, C = m->n_classes;
    if (m->d % 8 != 0 || h % 16 != 0 || h < 16 || h > 512 || (h > 256 && h % 256 != 0) || C < 1 || C > 16)
      return NGC_ERR_INVALID;
    rc = ensure_ws(p, ngc::mlp_scratch_bytes(k, m->rows_per_partition, m->d, h, C));
    if (rc != NGC_OK) return rc;
    long long ldG = 0;
    if ((rc = profile_mark(p, stream)) != NGC_OK) return rc;
    NGC_CUDA(p, ngc::launch_mlp_grad(k, m->rows_per_partition, m->d, h, C, static_cast<const float *>(X),
                                     static_cast<const int *>(y), static_cast<const float *>(theta),
                                     static_cast<unsigned char *>(p->ws), &G, &ldG, p->d_status, sms, stream,
                                     reinterpret_cast<ngc::DenseState **>(&p->dense_state)));
    if ((rc = profile_mark(p, stream)) != NGC_OK) return rc;
    out->ws = G;
    out->ld = ldG;
    out->launches = ngc::mlp_launch_count(h) - 1;
    return NGC_OK;
  }
  return NGC_ERR_INVALID;
}

int grad_encode_impl(ngc_plan_t *p, const ngc_model_t *m, const void *theta, const void *X, const void *y, int layer,
                     void *coded, void *cuda_stream, DecodeHook *hook) {
  if (hook) hook->fused = false;
  if (!p || !theta || !X || !y || !coded || layer < 0 || layer >= p->L) return NGC_ERR_INVALID;
  int rc = check_model(p, m);
  if (rc != NGC_OK) return rc;
  if (!aligned16(X) || !aligned16(coded) || !aligned16(theta)) return NGC_ERR_INVALID;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  rc = ensure_tables(p);
  if (rc != NGC_OK) return rc;
  const int cdt = ngc_coded_dtype(p, m);
  const ngc_level_t &lv = p->lv[layer];
  PartialGrads pg;
  if ((rc = partial_gradients(p, m, theta, X, y, p->n, stream, &pg)) != NGC_OK) return rc;
  if (hook && hook->after_grads) NGC_CUDA(p, cudaEventRecord(hook->after_grads, stream));
  if (m->kind == NGC_LSQ || m->kind == NGC_LOGISTIC) {
    NGC_CUDA(p, ngc::launch_combine_encode(pg.split, pg.ws, lv.d_coef, p->n, lv.s, m->d, coded, cdt, stream));
  } else {
    if ((rc = encode_dense(p, pg.split, pg.ws, pg.ld, lv, ngc_num_params(m), coded, cdt, stream, hook)) != NGC_OK)
      return rc;
  }
  p->launches += pg.launches + 1;
  return NGC_OK;
}

}  // namespace

extern "C" {

// ---- one problem sharded over several GPUs (Section II-C: the workers, each with its partitions, are independent)

int ngc_shard_gradients(ngc_plan_t *p, const ngc_model_t *m, const void *theta, const void *X_local, const void *y_local,
                        int n_local, float *G, int64_t ld, void *cuda_stream) {
  if (!p || !theta || !X_local || !y_local || !G || n_local < 1 || n_local > p->n) return NGC_ERR_INVALID;
  int rc = check_model(p, m);
  if (rc != NGC_OK) return rc;
  const int64_t l = ngc_num_params(m);
  if (ld < l || ld % 4 != 0 || !aligned16(X_local) || !aligned16(theta) || !aligned16(G)) return NGC_ERR_INVALID;
  if ((rc = ensure_tables(p)) != NGC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  PartialGrads pg;
  if ((rc = partial_gradients(p, m, theta, X_local, y_local, n_local, stream, &pg)) != NGC_OK) return rc;
  NGC_CUDA(p, ngc::launch_sum_slots(pg.split, n_local, pg.ws, pg.ld, l, G, ld, stream));
  p->launches += pg.launches + 1;
  return NGC_OK;
}

int ngc_shard_encode_decode(ngc_plan_t *p, const ngc_model_t *m, int layer, int first_worker, int n_local,
                            const float *G_window, int64_t ld, const int32_t *S, int nS, void *coded, void *partial,
                            void *cuda_stream) {
  if (!p || !G_window || !coded || !partial || layer < 0 || layer >= p->L) return NGC_ERR_INVALID;
  int rc = check_model(p, m);
  if (rc != NGC_OK) return rc;
  const ngc_level_t &lv = p->lv[layer];
  const int n = p->n, s = lv.s, rows = n_local + s;  // the shard's workers, then s rows that only pad the windows
  if (first_worker < 0 || first_worker >= n || n_local < 1 || n_local > n || rows > NGC_MAX_N) return NGC_ERR_INVALID;
  const int64_t l = ngc_num_params(m);
  if (ld < l || ld % 4 != 0 || !aligned16(G_window) || !aligned16(coded) || !aligned16(partial)) return NGC_ERR_INVALID;
  ngc::MaskArg mask;
  if ((rc = pack_set(p, layer, S, nS, mask.w)) != NGC_OK) return rc;
  if ((rc = ensure_tables(p)) != NGC_OK) return rc;
  if ((rc = ensure_batch(p, 1)) != NGC_OK) return rc;
  const size_t table = (size_t)NGC_MAX_N * (NGC_MAX_S + 1);
  if (!p->d_shard_coef) {
    NGC_CUDA(p, cudaMalloc(&p->d_shard_coef, (size_t)p->L * table * sizeof(double)));
    NGC_CUDA(p, cudaMalloc(&p->d_shard_a, (size_t)NGC_MAX_N * sizeof(double)));
    p->shard_key.assign((size_t)2 * p->L, -1);
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  double *d_coef = p->d_shard_coef + (size_t)layer * table;
  if (p->shard_key[2 * layer] != first_worker || p->shard_key[2 * layer + 1] != n_local) {
    // Rows first_worker .. first_worker + n_local - 1 of B (window form), then s all-zero rows: the encode kernels
    // index the partial gradients cyclically over `rows` entries, and only the zero rows ever wrap.  A rank asks
    // for the same shard in every iteration, so each level's table is uploaded once; when the shard does change,
    // work queued on the stream may still read the old table: wait for it first.
    p->shard_coef_host.assign((size_t)rows * (s + 1), 0.0);
    for (int r = 0; r < n_local; ++r) {
      const int i = (first_worker + r) % n;
      for (int t = 0; t <= s; ++t) p->shard_coef_host[(size_t)r * (s + 1) + t] = lv.coef[(size_t)i * (s + 1) + t];
    }
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    NGC_CUDA(p, cudaStreamIsCapturing(stream, &cap));
    if (cap != cudaStreamCaptureStatusNone) return NGC_ERR_INVALID;  // serve the shard once eagerly before capturing
    NGC_CUDA(p, cudaStreamSynchronize(stream));
    NGC_CUDA(p, cudaMemcpy(d_coef, p->shard_coef_host.data(), p->shard_coef_host.size() * sizeof(double),
                           cudaMemcpyHostToDevice));
    p->shard_key[2 * layer] = first_worker;
    p->shard_key[2 * layer + 1] = n_local;
  }
  const int cdt = ngc_coded_dtype(p, m);
  ngc::RowSplit split;
  split.T = rows; split.rows_g = 1; split.grid = rows; split.P = 1;
  NGC_CUDA(p, ngc::launch_encode_long(split, G_window, ld, d_coef, rows, s, l, coded, cdt, stream));
  // the decoding vector of the whole responsive set; this shard applies the weights of its own workers
  NGC_CUDA(p, ngc::launch_decode_solve(*p, layer, nullptr, mask, 1, p->d_a, p->d_resid, p->d_maxres, stream));
  NGC_CUDA(p, cudaMemsetAsync(p->d_shard_a, 0, (size_t)NGC_MAX_N * sizeof(double), stream));
  const int head = (first_worker + n_local <= n) ? n_local : n - first_worker;  // workers before the index wraps
  NGC_CUDA(p, cudaMemcpyAsync(p->d_shard_a, p->d_a + first_worker, (size_t)head * sizeof(double),
                              cudaMemcpyDeviceToDevice, stream));
  if (head < n_local)
    NGC_CUDA(p, cudaMemcpyAsync(p->d_shard_a + head, p->d_a, (size_t)(n_local - head) * sizeof(double),
                                cudaMemcpyDeviceToDevice, stream));
  if (cdt == NGC_F64)
    NGC_CUDA(p, ngc::launch_decode(coded, cdt, p->d_shard_a, rows, l, nullptr, stream, static_cast<double *>(partial)));
  else
    NGC_CUDA(p, ngc::launch_decode(coded, cdt, p->d_shard_a, rows, l, static_cast<float *>(partial), stream));
  p->launches += 3;
  return NGC_OK;
}

int ngc_prepare_data(ngc_plan_t *p, const ngc_model_t *m, const void *X, void *cuda_stream) {
  if (!p) return NGC_ERR_INVALID;
  int rc = check_model(p, m);
  if (rc != NGC_OK) return rc;
  if (m->kind != NGC_MLP) return NGC_OK;  // the other models read the data matrix as it is
  if (m->x_dtype != NGC_F32 || m->d % 8 != 0 || (X && !aligned16(X))) return NGC_ERR_INVALID;
  NGC_CUDA(p, ngc::prepare_mlp_data(reinterpret_cast<ngc::DenseState **>(&p->dense_state), p->k, m->rows_per_partition,
                                    m->d, static_cast<const float *>(X), static_cast<cudaStream_t>(cuda_stream)));
  if (X) p->launches += 1;
  return NGC_OK;
}

int ngc_shard_prepare_data(ngc_plan_t *p, const ngc_model_t *m, const void *X_local, int n_local, void *cuda_stream) {
  if (!p || n_local < 1 || n_local > p->n) return NGC_ERR_INVALID;
  int rc = check_model(p, m);
  if (rc != NGC_OK) return rc;
  if (m->kind != NGC_MLP) return NGC_OK;
  if (m->x_dtype != NGC_F32 || m->d % 8 != 0 || (X_local && !aligned16(X_local))) return NGC_ERR_INVALID;
  NGC_CUDA(p, ngc::prepare_mlp_data(reinterpret_cast<ngc::DenseState **>(&p->dense_state), n_local * (p->k / p->n),
                                    m->rows_per_partition, m->d, static_cast<const float *>(X_local),
                                    static_cast<cudaStream_t>(cuda_stream)));
  if (X_local) p->launches += 1;
  return NGC_OK;
}

int ngc_decode_vectors(ngc_plan_t *p, int layer, const int32_t *S, int nS, int batch, double *a_out,
                       double *resid_out) {
  if (!p || !S || !a_out || layer < 0 || layer >= p->L || batch < 1) return NGC_ERR_INVALID;
  std::vector<uint64_t> masks((size_t)batch * 2);
  for (int b = 0; b < batch; ++b) {
    const int rc = pack_set(p, layer, S + (size_t)b * nS, nS, &masks[2 * (size_t)b]);
    if (rc != NGC_OK) return rc;
  }
  int rc = ensure_tables(p);
  if (rc != NGC_OK) return rc;
  rc = ensure_batch(p, batch);
  if (rc != NGC_OK) return rc;
  NGC_CUDA(p, cudaMemcpy(p->d_masks, masks.data(), masks.size() * sizeof(uint64_t), cudaMemcpyHostToDevice));
  ngc::MaskArg none{{0, 0}};
  NGC_CUDA(p, ngc::launch_decode_solve(*p, layer, p->d_masks, none, batch, p->d_a, p->d_resid, nullptr, 0));
  p->launches += 1;
  NGC_CUDA(p, cudaMemcpy(a_out, p->d_a, (size_t)batch * p->n * sizeof(double), cudaMemcpyDeviceToHost));
  std::vector<double> res(batch);
  NGC_CUDA(p, cudaMemcpy(res.data(), p->d_resid, (size_t)batch * sizeof(double), cudaMemcpyDeviceToHost));
  int status = NGC_OK;
  for (int b = 0; b < batch; ++b) {
    if (resid_out) resid_out[b] = res[b];
    if (!(res[b] <= kResidualLimit)) status = NGC_ERR_SINGULAR;
  }
  return status;
}

int ngc_decode_vector(ngc_plan_t *p, int layer, const int32_t *S, int nS, double *a_out) {
  return ngc_decode_vectors(p, layer, S, nS, 1, a_out, nullptr);
}

int ngc_decode(ngc_plan_t *p, int layer, const int32_t *S, int nS, const void *coded, int coded_dtype, int64_t l,
               float *grad, void *cuda_stream) {
  if (!p || !coded || !grad || layer < 0 || layer >= p->L || l < 1) return NGC_ERR_INVALID;
  if (coded_dtype != NGC_F32 && coded_dtype != NGC_F64) return NGC_ERR_INVALID;
  if (!aligned16(coded)) return NGC_ERR_INVALID;
  ngc::MaskArg mask;
  int rc = pack_set(p, layer, S, nS, mask.w);
  if (rc != NGC_OK) return rc;
  rc = ensure_tables(p);
  if (rc != NGC_OK) return rc;
  rc = ensure_batch(p, 1);
  if (rc != NGC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  NGC_CUDA(p, ngc::launch_decode_solve(*p, layer, nullptr, mask, 1, p->d_a, p->d_resid, p->d_maxres, stream));
  NGC_CUDA(p, ngc::launch_decode(coded, coded_dtype, p->d_a, p->n, l, grad, stream));
  p->launches += 2;
  return NGC_OK;
}

// The decoding vector depends only on the responsive set, which is known before any gradient is:
// ngc_step solves it on a stream of the plan's own, under the gradient kernels, and the decode on the
// caller's stream waits for it.  The solve in turn waits for everything the caller's stream held when the
// step was entered (the decode of the step before reads the same vector).  Where the gradient kernel leaves no
// room on its SMs, the solve waits for that kernel instead and runs beside the small encode kernel.  A capturing
// stream takes the plain in-order path.
int ngc_step(ngc_plan_t *p, const ngc_model_t *m, const void *theta, const void *X, const void *y,
             const double *task_times, void *coded, float *grad, ngc_step_info_t *info, void *cuda_stream) {
  if (!p || !info) return NGC_ERR_INVALID;
  int rc = check_model(p, m);
  if (rc != NGC_OK) return rc;
  rc = ngc_select(p, task_times, info);
  if (rc != NGC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  NGC_CUDA(p, cudaStreamIsCapturing(stream, &cap));
  // A gradient CTA that fills its SM's register file would have to wait for the solve's block to leave
  // (and the solve is slow under a bandwidth-bound kernel): such models keep the in-order path.
  if (p->overlap_kind != m->kind || p->overlap_d != m->d || p->overlap_dtype != m->x_dtype) {
    p->overlap_kind = m->kind; p->overlap_d = m->d; p->overlap_dtype = m->x_dtype;
    p->overlap_ok = (m->kind == NGC_LSQ || m->kind == NGC_LOGISTIC) ? ngc::gemv_pair_leaves_room(*m) : true;
  }
  if (cap != cudaStreamCaptureStatusNone || !coded || !grad || !aligned16(coded)) {
    rc = ngc_grad_encode(p, m, theta, X, y, info->layer, coded, cuda_stream);
    if (rc != NGC_OK) return rc;
    return ngc_decode(p, info->layer, info->S, info->nS, coded, ngc_coded_dtype(p, m), ngc_num_params(m), grad,
                      cuda_stream);
  }
  ngc::MaskArg mask;
  rc = pack_set(p, info->layer, info->S, info->nS, mask.w);
  if (rc != NGC_OK) return rc;
  if ((rc = ensure_tables(p)) != NGC_OK) return rc;
  if ((rc = ensure_batch(p, 1)) != NGC_OK) return rc;
  if (!p->side_stream) {
    cudaStream_t s2;
    cudaEvent_t e1, e2, e3;
    NGC_CUDA(p, cudaStreamCreateWithFlags(&s2, cudaStreamNonBlocking));
    p->side_stream = s2;
    NGC_CUDA(p, cudaEventCreateWithFlags(&e1, cudaEventDisableTiming));
    p->ev_solved = e1;
    NGC_CUDA(p, cudaEventCreateWithFlags(&e2, cudaEventDisableTiming));
    p->ev_decoded = e2;
    NGC_CUDA(p, cudaEventCreateWithFlags(&e3, cudaEventDisableTiming));
    p->ev_grads = e3;
  }
  cudaStream_t side = static_cast<cudaStream_t>(p->side_stream);
  cudaEvent_t solved = static_cast<cudaEvent_t>(p->ev_solved), decoded = static_cast<cudaEvent_t>(p->ev_decoded);
  DecodeHook hook{solved, grad, false, nullptr};
  if (p->overlap_ok) {
    // Everything already queued on the caller's stream comes before the solve overwrites the vector: the decode
    // of the step before, but also a replayed graph whose captured steps recorded no event.
    NGC_CUDA(p, cudaEventRecord(decoded, stream));
    NGC_CUDA(p, cudaStreamWaitEvent(side, decoded, 0));
    NGC_CUDA(p, ngc::launch_decode_solve(*p, info->layer, nullptr, mask, 1, p->d_a, p->d_resid, p->d_maxres, side));
    NGC_CUDA(p, cudaEventRecord(solved, side));
  } else {
    // The gradient kernel fills its SMs: the solve waits for it on the side stream and runs beside the small
    // encode kernel instead of in line behind it.
    hook.after_grads = static_cast<cudaEvent_t>(p->ev_grads);
    hook.grad = nullptr;  // the vector is solved after the gradients: the decode stays a kernel of its own
  }
  // Dense models: the encode kernel forms the decoded gradient from the coded rows as it writes them.
  rc = grad_encode_impl(p, m, theta, X, y, info->layer, coded, cuda_stream, &hook);
  if (rc != NGC_OK) return rc;
  if (!p->overlap_ok) {
    // (the gradient kernels of this step come after the decode of the step before on the caller's stream, so the
    // vector is free by the time the event fires)
    NGC_CUDA(p, cudaStreamWaitEvent(side, hook.after_grads, 0));
    NGC_CUDA(p, ngc::launch_decode_solve(*p, info->layer, nullptr, mask, 1, p->d_a, p->d_resid, p->d_maxres, side));
    NGC_CUDA(p, cudaEventRecord(solved, side));
  }
  if (!hook.fused) {
    NGC_CUDA(p, cudaStreamWaitEvent(stream, solved, 0));
    NGC_CUDA(p, ngc::launch_decode(coded, ngc_coded_dtype(p, m), p->d_a, p->n, ngc_num_params(m), grad, stream));
    p->launches += 1;
  }
  p->launches += 1;  // the solve
  return NGC_OK;
}

int ngc_step_host(ngc_plan_t *p, const ngc_model_t *m, const float *theta, const void *X, const void *y,
                  const double *task_times, float *grad, ngc_step_info_t *info) {
  if (!p || !theta || !X || !y || !grad || !info) return NGC_ERR_INVALID;
  int rc = check_model(p, m);
  if (rc != NGC_OK) return rc;
  const int64_t l = ngc_num_params(m);
  const size_t xb = (size_t)p->k * m->rows_per_partition * m->d * (m->x_dtype == NGC_F32 ? 4 : 2);
  const size_t yb = (size_t)p->k * m->rows_per_partition * 4;
  const size_t cb = (size_t)p->n * l * (ngc_coded_dtype(p, m) == NGC_F64 ? 8 : 4);
  if ((rc = ensure_staging(p, &p->st_X, &p->st_X_bytes, xb)) != NGC_OK) return rc;
  if ((rc = ensure_staging(p, &p->st_y, &p->st_y_bytes, yb)) != NGC_OK) return rc;
  if ((rc = ensure_staging(p, &p->st_theta, &p->st_theta_bytes, (size_t)l * 4)) != NGC_OK) return rc;
  if ((rc = ensure_staging(p, &p->st_coded, &p->st_coded_bytes, cb)) != NGC_OK) return rc;
  if ((rc = ensure_staging(p, &p->st_grad, &p->st_grad_bytes, (size_t)l * 4)) != NGC_OK) return rc;
  cudaStream_t stream = 0;
  NGC_CUDA(p, cudaMemcpyAsync(p->st_theta, theta, (size_t)l * 4, cudaMemcpyHostToDevice, stream));
  NGC_CUDA(p, cudaMemcpyAsync(p->st_y, y, yb, cudaMemcpyHostToDevice, stream));
  NGC_CUDA(p, cudaMemcpyAsync(p->st_X, X, xb, cudaMemcpyHostToDevice, stream));
  rc = ngc_step(p, m, p->st_theta, p->st_X, p->st_y, task_times, p->st_coded, static_cast<float *>(p->st_grad), info,
                stream);
  if (rc != NGC_OK) return rc;
  NGC_CUDA(p, cudaMemcpyAsync(grad, p->st_grad, (size_t)l * 4, cudaMemcpyDeviceToHost, stream));
  NGC_CUDA(p, cudaStreamSynchronize(stream));
  return NGC_OK;
}

int ngc_latency_mc(ngc_plan_t *p, uint64_t seed, int64_t trials, double rho, double lambda, double p_fail,
                   double *latency_dev, int32_t *level_dev, void *cuda_stream) {
  if (!p || trials < 1 || !(rho >= 0.0) || !(lambda > 0.0) || !(p_fail >= 0.0 && p_fail <= 1.0)) return NGC_ERR_INVALID;
  if (!latency_dev && !level_dev) return NGC_ERR_INVALID;  // one of the two outputs may be left out
  NGC_CUDA(p, ngc::launch_latency_mc(*p, seed, trials, rho, lambda, p_fail, latency_dev, level_dev,
                                     static_cast<cudaStream_t>(cuda_stream)));
  p->launches += 1;
  return NGC_OK;
}

int ngc_gd_update(float *theta, const float *grad, int64_t l, float step, void *cuda_stream) {
  if (!theta || !grad || l < 1 || !(step == step)) return NGC_ERR_INVALID;
  return ngc::launch_gd_update(theta, grad, l, step, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? NGC_OK
                                                                                                            : NGC_ERR_CUDA;
}

size_t ngc_workspace_bytes(const ngc_plan_t *p) {
  if (!p) return 0;
  return p->ws_bytes + p->gpart_bytes + ngc::dense_state_bytes(static_cast<const ngc::DenseState *>(p->dense_state)) +
         p->st_X_bytes + p->st_y_bytes + p->st_theta_bytes + p->st_coded_bytes +
         p->st_grad_bytes;
}

int ngc_device_status(ngc_plan_t *p, double *residual_out) {
  if (!p) return NGC_ERR_INVALID;
  if (residual_out) *residual_out = 0.0;
  if (!p->tables_on_device) return NGC_OK;
  NGC_CUDA(p, cudaDeviceSynchronize());
  int st[2] = {0, 0};
  double mr = 0.0;
  NGC_CUDA(p, cudaMemcpy(st, p->d_status, sizeof(st), cudaMemcpyDeviceToHost));
  NGC_CUDA(p, cudaMemcpy(&mr, p->d_maxres, sizeof(mr), cudaMemcpyDeviceToHost));
  if (residual_out) *residual_out = mr;
  if (st[0] != 0) {  // reported once: the word is cleared so that later work on the plan is judged on its own
    NGC_CUDA(p, cudaMemset(p->d_status, 0, sizeof(int)));
    return NGC_ERR_TIMEOUT;
  }
  if (!(mr <= kResidualLimit)) return NGC_ERR_SINGULAR;
  return NGC_OK;
}

int ngc_selftest_wait_timeout(ngc_plan_t *p, int64_t limit_cycles, void *cuda_stream) {
  if (!p || limit_cycles < 1 || limit_cycles > 2000000000ll) return NGC_ERR_INVALID;
  const int rc = ensure_tables(p);
  if (rc != NGC_OK) return rc;
  NGC_CUDA(p, ngc::launch_wait_timeout(limit_cycles, p->d_status, static_cast<cudaStream_t>(cuda_stream)));
  p->launches += 1;
  return NGC_OK;
}

int ngc_dense_schedule(int batch, int m_blocks, int n_cols, int k_chunks, int max_pairs, int32_t *units_out, int cap,
                       int *n_units_out, int *n_pairs_out) {
  if (batch < 1 || m_blocks < 1 || n_cols < 1 || k_chunks < 1 || max_pairs < 1 || cap < 0 || !n_units_out ||
      !n_pairs_out || (cap > 0 && !units_out))
    return NGC_ERR_INVALID;
  static_assert(sizeof(int32_t) == sizeof(int), "unit rows are written as int");
  *n_units_out = ngc::wide_schedule_units(batch, m_blocks, n_cols, k_chunks, max_pairs,
                                          reinterpret_cast<int *>(units_out), cap, n_pairs_out);
  return NGC_OK;
}

int ngc_profile_enable(ngc_plan_t *p, int on) {
  if (!p) return NGC_ERR_INVALID;
  p->profiling = on != 0;
  return NGC_OK;
}

int ngc_profile_read(ngc_plan_t *p, double *ms_total, int64_t *launches) {
  if (!p || !ms_total || !launches) return NGC_ERR_INVALID;
  *ms_total = 0.0;
  *launches = 0;
  for (size_t i = 0; i + 1 < p->ev_used; i += 2) {
    cudaEvent_t a = static_cast<cudaEvent_t>(p->ev[i]), b = static_cast<cudaEvent_t>(p->ev[i + 1]);
    NGC_CUDA(p, cudaEventSynchronize(b));
    float ms = 0.f;
    NGC_CUDA(p, cudaEventElapsedTime(&ms, a, b));
    *ms_total += ms;
    *launches += 1;
  }
  p->ev_used = 0;
  return NGC_OK;
}

int ngc_last_cuda_error(const ngc_plan_t *p) { return p ? p->last_cuda : 0; }
int64_t ngc_launch_count(const ngc_plan_t *p) { return p ? p->launches : 0; }

}  // extern "C"
