// Internal plan layout shared by the host-side construction and the CUDA entry points.
#pragma once
#include <cstdint>
#include <vector>

#include "ngc.h"

struct ngc_level_t {
  int s = 0;                 // tolerance of this component code
  std::vector<double> coef;  // n x (s+1): row i = B[i, i..i+s mod n]
  std::vector<double> a0;    // n: a particular solution of B^T a = 1 (minimum norm)
  std::vector<double> N;     // n x s row-major: orthonormal basis of {v : B^T v = 0}
  double plan_residual = 0;  // max |B^T a0 - 1|, |B^T N| seen at construction
  // device copies (made on first GPU use)
  double *d_coef = nullptr, *d_a0 = nullptr, *d_N = nullptr;
};

struct ngc_plan_s {
  int n = 0, k = 0, q = 1, L = 0;
  uint64_t seed = 0;
  double gamma = 0, eps = 0;
  std::vector<int> levels;
  std::vector<ngc_level_t> lv;
  std::vector<int32_t> order;            // n x (s_L+1)
  std::vector<int32_t> tasks_per_layer;  // L
  int coded_dtype_override = -1;

  // device state
  int device = -1;
  bool tables_on_device = false;
  void *ws = nullptr;          // scratch for partial gradients / intermediates
  size_t ws_bytes = 0;
  double *d_a = nullptr;       // decode vectors, batch x n
  double *d_resid = nullptr;   // per-pattern residual, batch
  uint64_t *d_masks = nullptr; // batch x 2 words
  int a_batch_cap = 0;
  int *d_status = nullptr;     // [0] timeout flag, [1] scratch
  double *d_maxres = nullptr;  // largest residual seen by asynchronous decodes
  // sharded operation: coefficient rows and decoding weights of the workers one shard holds
  double *d_shard_coef = nullptr;  // per level: NGC_MAX_N x (NGC_MAX_S + 1), the rows of B of the shard last served
  double *d_shard_a = nullptr;     // NGC_MAX_N
  std::vector<int> shard_key;      // per level: {first_worker, n_local} of the table on the device, -1 = none
  std::vector<double> shard_coef_host;
  void *dense_state = nullptr; // ngc::DenseState*: cached tensor maps of the dense launchers, data prepared once
  void *d_gpart = nullptr;     // per-chunk partial decodes of the fused encode + decode (dense models)
  size_t gpart_bytes = 0;
  // ngc_step solves the decoding vector on a stream of its own while the gradients are computed
  void *side_stream = nullptr; // cudaStream_t, non-blocking
  void *ev_solved = nullptr;   // cudaEvent_t: d_a holds the vector of the current step
  void *ev_decoded = nullptr;  // cudaEvent_t: the last decode has read d_a
  void *ev_grads = nullptr;    // cudaEvent_t: the gradient kernels of the current step are done
  int overlap_kind = -1, overlap_d = -1, overlap_dtype = -1;  // model the answer below was taken for
  bool overlap_ok = false;     // the gradient kernel leaves room for the solve's warp on its SMs
  // staging for ngc_step_host
  void *st_X = nullptr, *st_y = nullptr, *st_theta = nullptr, *st_coded = nullptr, *st_grad = nullptr;
  size_t st_X_bytes = 0, st_y_bytes = 0, st_theta_bytes = 0, st_coded_bytes = 0, st_grad_bytes = 0;
  // optional event brackets around the dominant kernel
  bool profiling = false;
  std::vector<void *> ev;      // cudaEvent_t pairs, reused
  size_t ev_used = 0;
  int last_cuda = 0;
  int64_t launches = 0;
};

// host-side pieces (ngc_host.cpp)
int ngc_host_build_plan(ngc_plan_s *p);
