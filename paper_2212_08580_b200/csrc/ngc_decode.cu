// Main-node side of the nested gradient code:
//   * decoding vectors (Definition 1: supp(a) inside the responsive set S, a B = 1), one warp
//     per straggler pattern, fp64;
//   * the decode itself, g = sum_{i in S} a_i x_i (Section II-C), a bandwidth-bound weighted
//     reduction over the coded gradients.
#include "ngc_device.h"
#include "ngc_pdl.cuh"

namespace ngc {

namespace {

// ------------------------------------------------------------------------------------------
// Decoding vector for one pattern.  With a0 a particular solution of B^T a = 1 and N an
// orthonormal basis of {v : B^T v = 0} (both from the plan), every solution is a0 + N z; asking
// it to vanish on the s unused workers T gives the s x s system  N[T,:] z = -a0[T].  Solved by
// Gaussian elimination with partial pivoting, one matrix row per lane.
// ------------------------------------------------------------------------------------------
constexpr int kSolveWarps = 4;

// Shared memory of one warp: M[s][s+1], z[s], a[n] doubles, then the list of unused workers and the
// used flags.  Sized by the level, so that a single-pattern solve (one warp, about 2 KB) finds room
// on an SM beside a resident gradient CTA and can run under it.
__host__ __device__ inline size_t solve_warp_bytes(int n, int s) {
  const size_t dbl = (size_t)s * (s + 1) + s + n;
  const size_t tail = (size_t)s * sizeof(int) + (size_t)n;
  return dbl * sizeof(double) + ((tail + 7) & ~(size_t)7);
}

__global__ void __launch_bounds__(kSolveWarps * 32)
decode_solve_kernel(const uint64_t *__restrict__ masks, MaskArg one, int batch, int n, int s,
                    const double *__restrict__ a0, const double *__restrict__ Nmat, const double *__restrict__ coef,
                    double *__restrict__ a_out, double *__restrict__ resid_out, double *maxres) {
  pdl_sync();
  extern __shared__ __align__(16) unsigned char solve_smem[];
  const int warps = blockDim.x >> 5;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int b = blockIdx.x * warps + w;
  if (b >= batch) return;
  const int ldm = s + 1;
  double *M = reinterpret_cast<double *>(solve_smem + (size_t)w * solve_warp_bytes(n, s));  // [s][s+1]
  double *zs = M + (size_t)s * ldm;
  double *as = zs + s;
  int *tlist = reinterpret_cast<int *>(as + n);
  unsigned char *used = reinterpret_cast<unsigned char *>(tlist + s);
  uint64_t m0, m1;
  if (masks) { m0 = masks[2 * b]; m1 = masks[2 * b + 1]; }
  else { m0 = one.w[0]; m1 = one.w[1]; }

  if (lane == 0) {
    int kept = 0, nt = 0;
    for (int i = 0; i < n; ++i) {
      const bool in = ((i < 64 ? (m0 >> i) : (m1 >> (i - 64))) & 1ull) != 0;
      if (in && kept < n - s) { used[i] = 1; ++kept; }
      else { used[i] = 0; if (nt < s) tlist[nt] = i; ++nt; }
    }
  }
  __syncwarp();

  if (s > 0) {
    if (lane < s) {
      const int row = tlist[lane];
      for (int c = 0; c < s; ++c) M[(lane) * ldm + (c)] = Nmat[(size_t)row * s + c];
      M[(lane) * ldm + (s)] = -a0[row];
    }
    __syncwarp();
    for (int p = 0; p < s; ++p) {
      // pivot: largest magnitude in column p among rows >= p, smallest row on ties
      double v = (lane >= p && lane < s) ? fabs(M[(lane) * ldm + (p)]) : -1.0;
      int q = lane;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, v, off);
        const int oq = __shfl_xor_sync(0xffffffffu, q, off);
        if (ov > v || (ov == v && oq < q)) { v = ov; q = oq; }
      }
      if (q != p) {
        for (int c = lane; c <= s; c += 32) {
          const double tmp = M[(p) * ldm + (c)];
          M[(p) * ldm + (c)] = M[(q) * ldm + (c)];
          M[(q) * ldm + (c)] = tmp;
        }
      }
      __syncwarp();
      if (lane > p && lane < s) {
        const double f = M[(lane) * ldm + (p)] / M[(p) * ldm + (p)];
        for (int c = p + 1; c <= s; ++c) M[(lane) * ldm + (c)] -= f * M[(p) * ldm + (c)];
      }
      __syncwarp();
    }
    for (int p = s - 1; p >= 0; --p) {      // column-oriented back substitution
      if (lane == p) zs[p] = M[(p) * ldm + (s)] / M[(p) * ldm + (p)];
      __syncwarp();
      if (lane < p) M[(lane) * ldm + (s)] -= M[(lane) * ldm + (p)] * zs[p];
      __syncwarp();
    }
  }
  for (int i = lane; i < n; i += 32) {
    double v = 0.0;
    if (used[i]) {
      v = a0[i];
      for (int c = 0; c < s; ++c) v += Nmat[(size_t)i * s + c] * zs[c];
    }
    as[i] = v;
    a_out[(size_t)b * n + i] = v;
  }
  __syncwarp();
  // residual max_j |sum_i a_i B[i, j] - 1| over the cyclic windows
  double worst = 0.0;
  for (int j = lane; j < n; j += 32) {
    double acc = 0.0;
    for (int t = 0; t <= s; ++t) {
      int i = j - t;
      if (i < 0) i += n;
      acc += as[i] * coef[(size_t)i * (s + 1) + t];
    }
    const double r = fabs(acc - 1.0);
    worst = fmax(worst, isnan(r) ? (double)INFINITY : r);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) worst = fmax(worst, __shfl_xor_sync(0xffffffffu, worst, off));
  if (lane == 0) {
    if (resid_out) resid_out[b] = worst;
    if (maxres) atomicMax(reinterpret_cast<unsigned long long *>(maxres), (unsigned long long)__double_as_longlong(worst));
  }
}

// ------------------------------------------------------------------------------------------
// Weighted reduction.  A block owns 32*V consecutive parameters; its 8 warps take the rows of the
// coded matrix round-robin (lane = V consecutive parameters, 16-byte loads), zero weights skipped,
// and the 8 partial sums are added in warp order, so reruns give identical bits.
// ------------------------------------------------------------------------------------------
constexpr int kDecWarps = 8;

template <typename CT, int V>
__global__ void __launch_bounds__(kDecWarps * 32) decode_kernel(const CT *__restrict__ coded, const double *__restrict__ a,
                                                              int n, long long l, float *__restrict__ grad,
                                                              double *__restrict__ grad64) {
  pdl_sync();
  __shared__ double as[NGC_MAX_N];
  __shared__ double part[kDecWarps][32 * V];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < n; i += blockDim.x) as[i] = a[i];
  __syncthreads();
  const long long col = ((long long)blockIdx.x * 32 + lane) * V;
  double acc[V];
#pragma unroll
  for (int e = 0; e < V; ++e) acc[e] = 0.0;
  if (col < l) {
#pragma unroll 4
    for (int i = warp; i < n; i += kDecWarps) {
      const double ai = as[i];
      if (ai == 0.0) continue;
      const CT *src = coded + (size_t)i * l + col;
      alignas(16) CT v[V];
      if (V * sizeof(CT) == 16) *reinterpret_cast<uint4 *>(v) = __ldg(reinterpret_cast<const uint4 *>(src));
      else if (V * sizeof(CT) == 8) *reinterpret_cast<uint2 *>(v) = __ldg(reinterpret_cast<const uint2 *>(src));
      else v[0] = __ldg(src);
#pragma unroll
      for (int e = 0; e < V; ++e) acc[e] = fma(ai, (double)v[e], acc[e]);
    }
  }
#pragma unroll
  for (int e = 0; e < V; ++e) part[warp][lane * V + e] = acc[e];
  __syncthreads();
  for (int c = threadIdx.x; c < 32 * V; c += blockDim.x) {
    const long long gc = (long long)blockIdx.x * 32 * V + c;
    if (gc < l) {
      double sum = 0.0;
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) sum += part[w][c];
      if (grad64) grad64[gc] = sum;  // partial decode of one shard: added to the other shards' before rounding
      else grad[gc] = (float)sum;
    }
  }
}

// The same reduction for long gradients, where there are enough columns to fill the GPU without splitting
// the rows: one thread owns V consecutive parameters and walks the rows with a non-zero weight in
// index order (a compacted list in shared memory), several loads in flight, no exchange between threads.
template <typename CT, int V>
__global__ void __launch_bounds__(256) decode_flat_kernel(const CT *__restrict__ coded, const double *__restrict__ a,
                                                          int n, long long l, float *__restrict__ grad,
                                                          double *__restrict__ grad64) {
  pdl_sync();
  __shared__ double as[NGC_MAX_N];
  __shared__ double wt[NGC_MAX_N];
  __shared__ int row[NGC_MAX_N];
  __shared__ int count;
  for (int i = threadIdx.x; i < n; i += blockDim.x) as[i] = a[i];
  __syncthreads();
  if (threadIdx.x == 0) {
    int m = 0;
    for (int i = 0; i < n; ++i)
      if (as[i] != 0.0) { wt[m] = as[i]; row[m] = i; ++m; }
    count = m;
  }
  __syncthreads();
  const long long col = ((long long)blockIdx.x * 256 + threadIdx.x) * V;
  if (col >= l) return;
  const int m = count;
  double acc[V];
#pragma unroll
  for (int e = 0; e < V; ++e) acc[e] = 0.0;
#pragma unroll 8
  for (int t = 0; t < m; ++t) {
    const CT *src = coded + (size_t)row[t] * l + col;
    alignas(16) CT v[V];
    if (V * sizeof(CT) == 16) *reinterpret_cast<uint4 *>(v) = __ldg(reinterpret_cast<const uint4 *>(src));
    else if (V * sizeof(CT) == 8) *reinterpret_cast<uint2 *>(v) = __ldg(reinterpret_cast<const uint2 *>(src));
    else v[0] = __ldg(src);
    const double w = wt[t];
#pragma unroll
    for (int e = 0; e < V; ++e) acc[e] = fma(w, (double)v[e], acc[e]);
  }
  if (grad64) {
#pragma unroll
    for (int e = 0; e < V; ++e) grad64[col + e] = acc[e];
    return;
  }
  float *dst = grad + col;
  if (V == 4 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
    *reinterpret_cast<float4 *>(dst) = make_float4((float)acc[0], (float)acc[V > 1 ? 1 : 0], (float)acc[V > 2 ? 2 : 0], (float)acc[V > 3 ? 3 : 0]);
  } else if (V == 2 && (reinterpret_cast<uintptr_t>(dst) & 7u) == 0) {
    *reinterpret_cast<float2 *>(dst) = make_float2((float)acc[0], (float)acc[V > 1 ? 1 : 0]);
  } else {
#pragma unroll
    for (int e = 0; e < V; ++e) dst[e] = (float)acc[e];
  }
}

constexpr long long kDecodeFlatFrom = 1 << 16;  // parameters from which one thread per V columns fills the GPU

template <typename CT, int V>
cudaError_t run_decode(const void *coded, const double *a, int n, long long l, float *grad, double *grad64,
                       cudaStream_t stream) {
  if (l >= kDecodeFlatFrom) {
    const long long per_block = 256 * V;
    launch_k(decode_flat_kernel<CT, V>, (unsigned)((l + per_block - 1) / per_block), 256, 0, stream, 
        static_cast<const CT *>(coded), a, n, l, grad, grad64);
    return cudaGetLastError();
  }
  const long long per_block = 32 * V;
  const unsigned blocks = (unsigned)((l + per_block - 1) / per_block);
  launch_k(decode_kernel<CT, V>, blocks, kDecWarps * 32, 0, stream, static_cast<const CT *>(coded), a, n, l, grad,
           grad64);
  return cudaGetLastError();
}

__global__ void __launch_bounds__(256) gd_update_kernel(float *__restrict__ theta, const float *__restrict__ grad,
                                                        long long l, float step) {
  pdl_sync();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < l) theta[i] = fmaf(-step, grad[i], theta[i]);
}

}  // namespace

cudaError_t launch_gd_update(float *theta, const float *grad, long long l, float step, cudaStream_t stream) {
  launch_k(gd_update_kernel, (unsigned)((l + 255) / 256), 256, 0, stream, theta, grad, l, step);
  return cudaGetLastError();
}

cudaError_t launch_decode_solve(const ngc_plan_s &p, int layer, const uint64_t *masks_dev, MaskArg one, int batch,
                                double *a_dev, double *resid_dev, double *maxres_dev, cudaStream_t stream) {
  const ngc_level_t &lv = p.lv[layer];
  const int warps = (batch < kSolveWarps) ? batch : kSolveWarps;
  const unsigned blocks = (unsigned)((batch + warps - 1) / warps);
  const size_t smem = (size_t)warps * solve_warp_bytes(p.n, lv.s);  // at most 4 x 10.3 KB
  launch_k(decode_solve_kernel, blocks, warps * 32, smem, stream, masks_dev, one, batch, p.n, lv.s, lv.d_a0, lv.d_N,
                                                           lv.d_coef, a_dev, resid_dev, maxres_dev);
  return cudaGetLastError();
}

cudaError_t launch_decode(const void *coded, int coded_dtype, const double *a_dev, int n, long long l, float *grad,
                          cudaStream_t stream, double *grad64) {
  // widest vector that keeps every row 16- / 8-byte aligned
  if (coded_dtype == NGC_F64) {
    if (l % 2 == 0) return run_decode<double, 2>(coded, a_dev, n, l, grad, grad64, stream);
    return run_decode<double, 1>(coded, a_dev, n, l, grad, grad64, stream);
  }
  if (l % 4 == 0) return run_decode<float, 4>(coded, a_dev, n, l, grad, grad64, stream);
  if (l % 2 == 0) return run_decode<float, 2>(coded, a_dev, n, l, grad, grad64, stream);
  return run_decode<float, 1>(coded, a_dev, n, l, grad, grad64, stream);
}

}  // namespace ngc
