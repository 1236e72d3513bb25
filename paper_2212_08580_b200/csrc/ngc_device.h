// Launchers implemented in the .cu files; called by the C-ABI entry points in ngc_api.cu.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "ngc_internal.h"

namespace ngc {

// How the global row range [0, T) is cut into `grid` contiguous CTA ranges and how the
// per-CTA partial gradients of one partition group are laid out in the scratch buffer.
struct RowSplit {
  long long T;       // total rows = n_groups * rows_g
  long long rows_g;  // rows per partition group (one atomic task)
  int grid;          // CTAs; grid <= T so that no CTA range is empty
  int P;             // scratch slots per group = max number of CTAs touching one group
};

__host__ __device__ inline long long split_begin(const RowSplit &s, long long c) { return (c * s.T) / s.grid; }
// CTA whose range contains global row `row`.
__host__ __device__ inline int split_owner(const RowSplit &s, long long row) {
  return (int)(((row + 1) * s.grid - 1) / s.T);
}

RowSplit make_row_split(int n_groups, long long rows_g, int max_grid);

// Streaming GEMV pair (least squares / logistic): partial gradients of every CTA range
// into scratch `ws` laid out [group][slot][d].
cudaError_t launch_gemv_pair(const ngc_model_t &m, const RowSplit &split, const void *X, const float *y,
                             const float *theta, float *ws, int *status, cudaStream_t stream);

// Sums the scratch slots of each group (fixed order) and applies the sparse code rows:
// coded[i] = sum_t coef[i][t] * g_{(i+t) mod n}.
cudaError_t launch_combine_encode(const RowSplit &split, const float *ws, const double *d_coef, int n, int s,
                                  int d, void *coded, int coded_dtype, cudaStream_t stream);

struct MaskArg {
  uint64_t w[2];
};
// Decoding vectors: one warp per pattern.  masks_dev == nullptr -> single pattern `one`.
cudaError_t launch_decode_solve(const ngc_plan_s &p, int layer, const uint64_t *masks_dev, MaskArg one, int batch,
                                double *a_dev, double *resid_dev, double *maxres_dev, cudaStream_t stream);

// g = sum_i a_i coded[i], a read from device memory (zeros skipped).  With grad64 the sum is written there
// unrounded instead of to grad (the partial decode of one shard of the workers).
cudaError_t launch_decode(const void *coded, int coded_dtype, const double *a_dev, int n, long long l, float *grad,
                          cudaStream_t stream, double *grad64 = nullptr);

// G_out[g][c] = sum over the scratch slots of group g (fp64, slot order), c < l: the partial gradients themselves,
// for a caller that exchanges them (sharded operation).  ws is [group][slot][ld_ws], G_out [group][ld_out].
cudaError_t launch_sum_slots(const RowSplit &split, int n_groups, const float *ws, long long ld_ws, long long l,
                             float *G_out, long long ld_out, cudaStream_t stream);

// True when an SM that holds a CTA of the gradient kernel chosen for `m` can still take a one-warp block.
bool gemv_pair_leaves_room(const ngc_model_t &m);

// Same encode for long gradients (dense models): every partial gradient is read once, windows live in
// registers.  ws is [group][slot][ld_ws] fp32, ld_ws a multiple of 4 and >= d.
// With `dec` (and a window that fits the register ring) the decode rides along: the kernel also forms
// grad = sum_i a[i] * coded[i] from the values it has just produced, through `gpart` (kEncodeMaxChunks x d
// doubles of scratch) when the workers are cut into several chunks; *fused tells whether it did.
constexpr int kEncodeMaxChunks = 16;
struct EncodeDecodeArgs {
  const double *a;  // decoding vector on the device, n weights, zero outside the responsive set
  double *gpart;
  float *grad;
  bool *fused;
  int *sum_launches;  // out: 1 when the chunk sum ran as a kernel of its own (more than one worker chunk), else 0
};
cudaError_t launch_encode_long(const RowSplit &split, const float *ws, long long ld_ws, const double *d_coef, int n,
                               int s, long long d, void *coded, int coded_dtype, cudaStream_t stream,
                               const EncodeDecodeArgs *dec = nullptr);

// Per-plan state of the dense launchers (created on first use): tensor maps and derived sizes of the last
// problem, so that a repeated call encodes nothing on the host, and the data prepared once for the MLP.
struct DenseState;
void dense_state_free(DenseState *st);
size_t dense_state_bytes(const DenseState *st);  // device memory it owns

// MLP (one hidden ReLU layer, softmax cross-entropy) partial gradients on the tensor cores (X fp32):
// G[k][*G_ld] fp32 inside `scratch`, each row holding [dW1, db1, dW2, db2].
size_t mlp_scratch_bytes(int k, int rows, int d, int hidden, int C);
int mlp_launch_count(int hidden);  // kernels one gradient + encode call launches
cudaError_t launch_mlp_grad(int k, int rows, int d, int hidden, int C, const float *X, const int *y, const float *theta,
                            unsigned char *scratch, float **G_out, long long *G_ld, int *status, int sms,
                            cudaStream_t stream, DenseState **state);
// bf16 copy [X 1] of the MLP's data matrix, made once and used by every later launch_mlp_grad on the same X
// (Section II-C: the data is assigned before training starts); X == nullptr drops it.
cudaError_t prepare_mlp_data(DenseState **state, int k, int rows, int d, const float *X, cudaStream_t stream);

// Softmax-regression partial gradients on the tensor cores (X bf16): G[k][d*C] fp32 inside `scratch`.
size_t softmax_scratch_bytes(int k, int rows, int d, int C);
cudaError_t launch_softmax_grad(int k, int rows, int d, int C, const void *X, const int *y, const float *W,
                                unsigned char *scratch, float **G_out, int *status, int sms, cudaStream_t stream,
                                DenseState **state);

// Host only: how the wide backward contraction (D^T = A^T B, M blocks of 256, N passes of 512 columns, some cut in
// halves) splits a problem into units and deals them to `max_pairs` CTA pairs; see ngc_dense_schedule in ngc.h.
int wide_schedule_units(int batch, int m_tiles, int n_total, int num_k, int max_pairs, int *units, int cap,
                        int *pairs_out);

// Monte Carlo of the stopping rule (Section IV): latency (gamma + eps + decode instant, +inf if never) and
// chosen level (-1 if none) of `trials` seeded straggler patterns, into device buffers.
cudaError_t launch_latency_mc(const ngc_plan_s &plan, uint64_t seed, long long trials, double shift, double rate,
                              double p_fail, double *latency_dev, int *level_dev, cudaStream_t stream);

// theta <- theta - step * grad (Eq. 1).
cudaError_t launch_gd_update(float *theta, const float *grad, long long l, float step, cudaStream_t stream);

// One warp waits at most `limit_cycles` SM cycles on a barrier nobody arrives on, then sets *status to 1.
cudaError_t launch_wait_timeout(long long limit_cycles, int *status, cudaStream_t stream);

int device_sm_count();

}  // namespace ngc
