// ngc_grad_encode_static: the least-squares / logistic gradient + encode for callers that must not
// allocate device memory.
//
// Who needs this: a host program whose device memory is owned entirely by its own allocator (a
// framework pool that has reserved the whole GPU, so that a raw cudaMalloc fails or fragments the
// pool), and a latency-critical loop that cannot afford the device-wide synchronisation a
// cudaMalloc / cudaFree may imply in the middle of an iteration.  ngc_grad_encode itself needs
// scratch for the per-CTA partial gradients and device copies of the code coefficients, which it
// takes from cudaMalloc through the plan.  Here both live in one fixed array that is part of the
// library image: every GPU that loads the library holds NGC_STATIC_SCRATCH_BYTES of it until the
// process exits.  Nothing in this file allocates or frees device memory.
#include <mutex>

#include "ngc_device.h"

namespace {

constexpr size_t kHeaderBytes = 256;                                                   // status word
constexpr size_t kCoefBytes = (size_t)NGC_MAX_N * (NGC_MAX_S + 1) * sizeof(double);    // 33 792
constexpr size_t kPartialBytes = NGC_STATIC_SCRATCH_BYTES - kHeaderBytes - kCoefBytes;  // 8 MiB

static_assert(kCoefBytes % 256 == 0, "coefficient block keeps the partials 256-byte aligned");

// [status | coefficients of the requested component code | per-CTA partial gradients]
static __device__ __align__(256) unsigned char ngc_static_scratch[NGC_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char *g_base[kMaxDevices] = {};  // device address of the array, per device

// The array's name is only a handle in host code; its device address has to be asked for, once per
// device, with that device current.
int scratch_base(unsigned char **out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NGC_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_base[dev]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, ngc_static_scratch) != cudaSuccess || !ptr) return NGC_ERR_CUDA;
    g_base[dev] = static_cast<unsigned char *>(ptr);
  }
  *out = g_base[dev];
  return NGC_OK;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int ngc_grad_encode_static(const ngc_plan_t *p, const ngc_model_t *m, const void *theta, const void *X,
                                      const void *y, int layer, void *coded, int32_t *status_dev, void *cuda_stream) {
  if (!p || !m || !theta || !X || !y || !coded || layer < 0 || layer >= p->L) return NGC_ERR_INVALID;
  if (m->kind != NGC_LSQ && m->kind != NGC_LOGISTIC) return NGC_ERR_INVALID;
  if (m->x_dtype != NGC_F32 && m->x_dtype != NGC_BF16) return NGC_ERR_INVALID;
  if (m->rows_per_partition < 1 || m->d < 1) return NGC_ERR_INVALID;
  const int vec = (m->x_dtype == NGC_F32) ? 4 : 8;
  if (m->d % vec != 0 || m->d / vec > 4 * 512) return NGC_ERR_INVALID;
  if (!aligned16(X) || !aligned16(coded) || !aligned16(theta)) return NGC_ERR_INVALID;
  const int sms = ngc::device_sm_count();
  if (sms <= 0) return NGC_ERR_CUDA;
  const ngc::RowSplit split = ngc::make_row_split(p->n, (long long)p->q * m->rows_per_partition, sms);
  const size_t need = (size_t)p->n * split.P * m->d * sizeof(float);
  if (need > kPartialBytes) return NGC_ERR_TOO_LARGE;  // n * slots * d floats must fit the fixed array

  unsigned char *base = nullptr;
  const int rc = scratch_base(&base);
  if (rc != NGC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int *status = status_dev ? status_dev : reinterpret_cast<int *>(base);
  double *coef = reinterpret_cast<double *>(base + kHeaderBytes);
  float *partials = reinterpret_cast<float *>(base + kHeaderBytes + kCoefBytes);
  const ngc_level_t &lv = p->lv[layer];

  // The array keeps whatever the previous call left.  The status word must start at zero; the
  // coefficients are overwritten; every partial-gradient slot that is read is written first.
  if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return NGC_ERR_CUDA;
  if (cudaMemcpyAsync(coef, lv.coef.data(), lv.coef.size() * sizeof(double), cudaMemcpyHostToDevice, stream) !=
      cudaSuccess)
    return NGC_ERR_CUDA;
  if (ngc::launch_gemv_pair(*m, split, X, static_cast<const float *>(y), static_cast<const float *>(theta), partials,
                            status, stream) != cudaSuccess)
    return NGC_ERR_CUDA;
  const int cdt = ngc_coded_dtype(p, m);
  if (ngc::launch_combine_encode(split, partials, coef, p->n, lv.s, m->d, coded, cdt, stream) != cudaSuccess)
    return NGC_ERR_CUDA;
  return NGC_OK;
}
