// Streaming GEMV pair for the least-squares and logistic partial gradients
// (Section II-C: g_j = sum over the rows of partition j of the per-sample loss gradient):
//     z = X_j theta,   r = act(z) - y_j,   g_j = X_j^T r
// fused so that every row of the data matrix is read from device memory exactly once.
//
// One persistent CTA per SM owns a contiguous range of the global row space.  Row tiles
// are brought into shared memory by bulk asynchronous copies (TMA, mbarrier completion)
// several stages ahead; every thread owns a fixed set of 16-byte column vectors, keeps
// theta and its slice of the gradient in registers, pulls its slice of the tile into
// registers once and uses it twice (dot product, then rank-1 update).  Row dot products
// are reduced with warp shuffles plus one shared-memory exchange per tile.
#include <cuda_bf16.h>

#include "ngc_device.h"
#include "ngc_pdl.cuh"
#include "ngc_f32x2.cuh"

namespace ngc {

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxStages = 8;
constexpr int kSmemReserve = 2048;       // barriers + reduction exchange + flags
constexpr int kSmemMax = 232448;         // 227 KB opt-in limit per CTA
constexpr long long kWaitCycles = 4000000000ll;

struct GemvParams {
  const unsigned char *X;
  const float *y;
  const float *theta;
  float *ws;
  int *status;
  RowSplit split;
  int d;
  int row_bytes;
  int stage_bytes;
  int stages;
  int act;  // 0: residual z - y (least squares), 1: sigmoid(z) - y (logistic)
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kWaitCycles SM cycles and reports failure instead of hanging.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > kWaitCycles) return false;
  }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

template <typename XT>
struct Vec;
template <>
struct Vec<float> {
  static constexpr int N = 4;  // elements per 16-byte vector
  __device__ static __forceinline__ void unpack(const uint4 &u, f32x2 (&f)[2]) {
    f[0] = pack2(__uint_as_float(u.x), __uint_as_float(u.y));
    f[1] = pack2(__uint_as_float(u.z), __uint_as_float(u.w));
  }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void unpack(const uint4 &u, f32x2 (&f)[4]) {
    f[0] = pack2(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
    f[1] = pack2(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
    f[2] = pack2(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u));
    f[3] = pack2(__uint_as_float(u.w << 16), __uint_as_float(u.w & 0xffff0000u));
  }
};

// Walks the tiles of one CTA range: at most R rows, never crossing a partition-group boundary.  Positions are
// kept relative to the first row of the range (32 bits: a range is the 148th part of the data), the absolute
// 64-bit row index is formed only where an address is.
struct TileWalk {
  long long base;
  int cur, end, seg_end, rows_g;
  int group;
  __device__ __forceinline__ void init(long long b, long long e, long long rg) {
    base = b; cur = 0; end = (int)(e - b); rows_g = (int)rg;
    group = (int)(b / rg);
    const long long se = (long long)(group + 1) * rg - b;
    seg_end = se < (long long)end ? (int)se : end;
  }
  __device__ __forceinline__ bool done() const { return cur >= end; }
  // returns the tile starting at `cur`; seg_last = it closes this CTA's piece of partition group `g`
  __device__ __forceinline__ void next(int R, long long &row0, int &nrows, bool &seg_last, int &g) {
    int e = cur + R;
    if (e > seg_end) e = seg_end;
    row0 = base + cur;
    nrows = e - cur;
    g = group;
    seg_last = (e == seg_end);
    cur = e;
    if (seg_last) {
      ++group;
      seg_end = (seg_end > end - rows_g) ? end : seg_end + rows_g;
    }
  }
};

// Sum over the 32 lanes of R per-lane values with R/2 + ... + 1 + log2(32/R) shuffles: at each of the
// first log2(R) steps a lane hands half of its values to its partner and keeps the other half.
// Afterwards lane l holds the full sum of row  bitrev-free index  (l >> (5 - log2 R)).
template <int R>
__device__ __forceinline__ float warp_reduce_rows(float (&v)[R], int lane) {
  int width = 16;
#pragma unroll
  for (int n = R; n > 1; n >>= 1) {
    const bool upper = (lane & width) != 0;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const float send = upper ? v[i] : v[i + n / 2];
      const float keep = upper ? v[i + n / 2] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, width);
    }
    width >>= 1;
  }
  float x = v[0];
#pragma unroll
  for (; width > 0; width >>= 1) x += __shfl_xor_sync(0xffffffffu, x, width);
  return x;
}

template <int R>
struct Log2;
template <> struct Log2<2> { static constexpr int v = 1; };
template <> struct Log2<4> { static constexpr int v = 2; };
template <> struct Log2<8> { static constexpr int v = 3; };

template <typename XT, int VPT, int R>
__global__ void __launch_bounds__(kThreads, 1) gemv_pair_kernel(const GemvParams p) {
  pdl_sync();
  constexpr int VN = Vec<XT>::N;
  constexpr int VH = VN / 2;  // packed pairs per vector
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *tiles = smem;
  unsigned char *tail = smem + (size_t)p.stages * p.stage_bytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(tail);        // kMaxStages
  float *red = reinterpret_cast<float *>(tail + 128);         // [R][kWarps] per-warp partial dot products
  float *resv = red + 2 * R * kWarps;                         // [R] residuals of the tile's rows (behind two red buffers)
  volatile int *abort_flag = reinterpret_cast<volatile int *>(resv + R);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nv = p.d / VN;  // 16-byte vectors per row

  if (tid == 0) {
    for (int s = 0; s < p.stages; ++s) mbar_init(smem_u32(&bars[s]), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const long long rb = split_begin(p.split, blockIdx.x), re = split_begin(p.split, blockIdx.x + 1);
  TileWalk prod, cons;
  prod.init(rb, re, p.split.rows_g);
  cons.init(rb, re, p.split.rows_g);
  int issued = 0;        // tiles issued by thread 0
  int issue_stage = 0;

  auto issue = [&]() {
    long long row0; int nrows, g; bool last;
    prod.next(R, row0, nrows, last, g);
    const uint32_t bar = smem_u32(&bars[issue_stage]);
    const uint32_t bytes = (uint32_t)nrows * (uint32_t)p.row_bytes;
    mbar_expect_tx(bar, bytes);
    bulk_g2s(smem_u32(tiles + (size_t)issue_stage * p.stage_bytes), p.X + (size_t)row0 * p.row_bytes, bytes, bar);
    ++issued;
    if (++issue_stage == p.stages) issue_stage = 0;
  };
  if (tid == 0)
    for (int s = 0; s < p.stages - 1 && !prod.done(); ++s) issue();

  // theta slice and gradient accumulators of this thread, as packed pairs
  f32x2 th[VPT][VH], acc[VPT][VH];
  bool vok[VPT];
#pragma unroll
  for (int c = 0; c < VPT; ++c) {
    const int v = tid + c * kThreads;
    vok[c] = v < nv;
#pragma unroll
    for (int e = 0; e < VH; ++e) {
      const float2 t2 = vok[c] ? __ldg(reinterpret_cast<const float2 *>(p.theta) + (size_t)v * VH + e)
                               : make_float2(0.f, 0.f);
      th[c][e] = pack2(t2.x, t2.y);
      acc[c][e] = pack2(0.f, 0.f);
    }
  }

  const uint32_t tiles_u32 = smem_u32(tiles) + (uint32_t)tid * 16u;
  int t = 0, st = 0;
  uint32_t parity = 0;
  bool failed = false;
  while (!cons.done()) {
    if (tid == 0 && !prod.done()) issue();  // refills the stage every thread left before the last barrier
    long long row0; int nrows, g; bool seg_last;
    cons.next(R, row0, nrows, seg_last, g);
    // the warps that will finish the row sums fetch the labels early
    float yrow = 0.f;
    if (R == 2) {
      if ((lane >> 4) < nrows) yrow = __ldg(p.y + row0 + (lane >> 4));
    } else if (warp < R && lane == 0 && warp < nrows) {
      yrow = __ldg(p.y + row0 + warp);
    }

    if (!mbar_wait(smem_u32(&bars[st]), parity)) {
      failed = true;
      *abort_flag = 1;
    }
    const uint32_t tile = tiles_u32 + (uint32_t)st * (uint32_t)p.stage_bytes;
    uint4 xr[R][VPT];
    float pd[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      f32x2 d2 = pack2(0.f, 0.f);
#pragma unroll
      for (int c = 0; c < VPT; ++c) {
        if (vok[c] && r < nrows)
          xr[r][c] = lds128(tile + (uint32_t)r * (uint32_t)p.row_bytes + (uint32_t)c * (kThreads * 16));
        else
          xr[r][c] = make_uint4(0u, 0u, 0u, 0u);
        f32x2 f[VH];
        Vec<XT>::unpack(xr[r][c], f);
#pragma unroll
        for (int e = 0; e < VH; ++e) fma2(d2, f[e], th[c][e]);
      }
      float lo, hi;
      unpack2(d2, lo, hi);
      pd[r] = lo + hi;
    }
    const float rowsum = warp_reduce_rows<R>(pd, lane);
    float res_r[R];
    if (R == 2) {
      // Two rows per tile: one barrier.  Every warp adds up the 16 per-warp parts of both rows itself (lanes 0-15
      // row 0, lanes 16-31 row 1) from a buffer that alternates with the tile's parity, so nobody waits for two
      // finishing warps and a second barrier.
      float *rb = red + (t & 1) * (R * kWarps);
      if ((lane & 15) == 0) rb[(lane >> 4) * kWarps + warp] = rowsum;
      __syncthreads();
      if (*abort_flag) break;
      float z = rb[lane];  // kWarps == 16: element (lane >> 4) * kWarps + (lane & 15)
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
      float res = (p.act ? 1.f / (1.f + expf(-z)) : z) - yrow;
      if ((lane >> 4) >= nrows) res = 0.f;
      res_r[0] = __shfl_sync(0xffffffffu, res, 0);
      res_r[R - 1] = __shfl_sync(0xffffffffu, res, 16);
    } else {
      if ((lane & (31 >> Log2<R>::v)) == 0) red[(lane >> (5 - Log2<R>::v)) * kWarps + warp] = rowsum;
      __syncthreads();
      if (warp < R) {  // warp r finishes row r: sum over the kWarps partials, then the residual
        float z = (lane < kWarps) ? red[warp * kWarps + lane] : 0.f;
#pragma unroll
        for (int off = kWarps / 2; off > 0; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
        if (lane == 0) {
          // (one code path for both activations: as two template instances the least-squares one, although the
          // simpler, was compiled with spills at the 128-register cap of the widest bf16 shape)
          const float res = (p.act ? 1.f / (1.f + expf(-z)) : z) - yrow;
          resv[warp] = (warp < nrows) ? res : 0.f;
        }
      }
      __syncthreads();
      if (*abort_flag) break;
#pragma unroll
      for (int r = 0; r < R; ++r) res_r[r] = resv[r];
    }
    if (sizeof(XT) == 2) {
      // keep the packed words, not their unpacked copies, live across the barriers
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < VPT; ++c)
          asm volatile("" : "+r"(xr[r][c].x), "+r"(xr[r][c].y), "+r"(xr[r][c].z), "+r"(xr[r][c].w));
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const float res = res_r[r];
      const f32x2 res2 = pack2(res, res);
#pragma unroll
      for (int c = 0; c < VPT; ++c) {
        f32x2 f[VH];
        Vec<XT>::unpack(xr[r][c], f);
#pragma unroll
        for (int e = 0; e < VH; ++e) fma2(acc[c][e], res2, f[e]);
      }
    }
    if (seg_last) {
      const int piece = (int)blockIdx.x - split_owner(p.split, (long long)g * p.split.rows_g);
      float *dst = p.ws + ((size_t)g * p.split.P + piece) * p.d + (size_t)tid * VN;
#pragma unroll
      for (int c = 0; c < VPT; ++c) {
        if (vok[c]) {
#pragma unroll
          for (int e = 0; e < VH; e += 2) {
            float4 o;
            unpack2(acc[c][e], o.x, o.y);
            unpack2(acc[c][e + 1], o.z, o.w);
            *reinterpret_cast<float4 *>(dst + (size_t)c * (kThreads * VN) + e * 2) = o;
          }
        }
#pragma unroll
        for (int e = 0; e < VH; ++e) acc[c][e] = pack2(0.f, 0.f);
      }
    }
    ++t;
    if (++st == p.stages) { st = 0; parity ^= 1u; }
  }
  if (failed) atomicExch(p.status, 1);
  if (*abort_flag && tid == 0) {
    // drain copies that are still in flight before the CTA (and its shared memory) goes away
    for (int u = t; u < issued; ++u) mbar_wait(smem_u32(&bars[u % p.stages]), (uint32_t)((u / p.stages) & 1));
  }
}

template <typename XT, int VPT, int R>
cudaError_t launch_one(const GemvParams &p, cudaStream_t stream) {
  const size_t smem = (size_t)p.stages * p.stage_bytes + kSmemReserve;
  auto kern = gemv_pair_kernel<XT, VPT, R>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  launch_k(kern, p.split.grid, kThreads, smem, stream, p);
  return cudaGetLastError();
}

// Whether one more small block (a warp or two, a few KB of shared memory) still fits on an SM that
// holds a CTA of this kernel: registers are what runs out first (512 threads x 128 registers fill the file).
template <typename XT, int VPT, int R>
bool room_beside(const GemvParams &p) {
  cudaFuncAttributes attr;
  if (cudaFuncGetAttributes(&attr, gemv_pair_kernel<XT, VPT, R>) != cudaSuccess) return false;
  const size_t smem = (size_t)p.stages * p.stage_bytes + kSmemReserve;
  return (size_t)attr.numRegs * kThreads + 64 * 64 <= 65536 && smem + 16384 <= 233472;
}

template <typename XT>
cudaError_t launch_shape(GemvParams &p, cudaStream_t stream, bool *room = nullptr) {
  const int nv = p.d / Vec<XT>::N;
  int vpt = (nv + kThreads - 1) / kThreads;
  int R;
  if (vpt <= 1) { vpt = 1; R = 8; }
  else if (vpt == 2) { R = 4; }
  else if (vpt <= 4) { vpt = 4; R = 2; }
  else return cudaErrorInvalidValue;
  p.stage_bytes = R * p.row_bytes;
  int stages = (kSmemMax - kSmemReserve) / p.stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return cudaErrorInvalidValue;
  p.stages = stages;
  if (room) {  // query only, nothing is launched
    *room = (vpt == 1) ? room_beside<XT, 1, 8>(p) : (vpt == 2) ? room_beside<XT, 2, 4>(p) : room_beside<XT, 4, 2>(p);
    return cudaSuccess;
  }
  if (vpt == 1) return launch_one<XT, 1, 8>(p, stream);
  if (vpt == 2) return launch_one<XT, 2, 4>(p, stream);
  return launch_one<XT, 4, 2>(p, stream);
}

}  // namespace

RowSplit make_row_split(int n_groups, long long rows_g, int max_grid) {
  RowSplit s;
  s.T = (long long)n_groups * rows_g;
  s.rows_g = rows_g;
  s.grid = (int)(s.T < max_grid ? s.T : max_grid);
  int P = 1;
  for (int g = 0; g < n_groups; ++g) {
    const int c0 = split_owner(s, g * rows_g), c1 = split_owner(s, (g + 1) * rows_g - 1);
    if (c1 - c0 + 1 > P) P = c1 - c0 + 1;
  }
  s.P = P;
  return s;
}

cudaError_t launch_gemv_pair(const ngc_model_t &m, const RowSplit &split, const void *X, const float *y,
                             const float *theta, float *ws, int *status, cudaStream_t stream) {
  GemvParams p;
  p.X = static_cast<const unsigned char *>(X);
  p.y = y;
  p.theta = theta;
  p.ws = ws;
  p.status = status;
  p.split = split;
  p.d = m.d;
  p.act = (m.kind == NGC_LOGISTIC) ? 1 : 0;
  if (m.x_dtype == NGC_F32) {
    p.row_bytes = m.d * 4;
    return launch_shape<float>(p, stream);
  }
  p.row_bytes = m.d * 2;
  return launch_shape<__nv_bfloat16>(p, stream);
}

bool gemv_pair_leaves_room(const ngc_model_t &m) {
  GemvParams p;
  p.d = m.d;
  p.row_bytes = m.d * (m.x_dtype == NGC_F32 ? 4 : 2);
  p.act = (m.kind == NGC_LOGISTIC) ? 1 : 0;
  bool room = false;
  const cudaError_t e = (m.x_dtype == NGC_F32) ? launch_shape<float>(p, 0, &room) : launch_shape<__nv_bfloat16>(p, 0, &room);
  return e == cudaSuccess && room;
}

// ---------------------------------------------------------------------------------------------
// Combine + encode: G[j] = sum of the scratch slots of group j (fp64, fixed order), then the sparse
// code rows x_i = sum_t B[i, i+t] g_{i+t}  (Section II-C, X = B G with the cyclic supports of Lemma 1).
// A block owns 128 columns x 8 workers; its 8 warps split the group sums and then the workers, each
// lane carrying 4 consecutive columns (16-byte loads of the fp32 partials).
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kEncCols = 128;  // columns per block
constexpr int kEncWarps = 8;

template <typename CT>
__global__ void __launch_bounds__(kEncWarps * 32)
combine_encode_kernel(const RowSplit split, const float *__restrict__ ws, const double *__restrict__ coef, int n, int s,
                      int d, CT *__restrict__ coded, int kEncRows /* workers per block */) {
  pdl_sync();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int held = min(kEncRows + s, n);
  double *Gs = reinterpret_cast<double *>(smem_raw);            // [held][kEncCols]
  double *cf = Gs + (size_t)held * kEncCols;                    // [kEncRows][s+1]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int col = blockIdx.x * kEncCols + lane * 4;
  const int i0 = blockIdx.y * kEncRows;
  const int ni = min(kEncRows, n - i0);
  for (int e = tid; e < ni * (s + 1); e += kEncWarps * 32) cf[e] = coef[(size_t)i0 * (s + 1) + e];
  const int ng = min(ni + s, n);  // groups i0 .. i0+ng-1 (mod n) are needed
  if (col < d) {
    for (int u = warp; u < ng; u += kEncWarps) {
      const int g = (i0 + u) % n;
      const int c0 = split_owner(split, (long long)g * split.rows_g);
      const int c1 = split_owner(split, (long long)(g + 1) * split.rows_g - 1);
      const float *src = ws + ((size_t)g * split.P) * d + col;
      double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
#pragma unroll 4
      for (int pce = 0; pce <= c1 - c0; ++pce) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(src + (size_t)pce * d));
        s0 += (double)v.x; s1 += (double)v.y; s2 += (double)v.z; s3 += (double)v.w;
      }
      double *dst = Gs + u * kEncCols + lane * 4;
      dst[0] = s0; dst[1] = s1; dst[2] = s2; dst[3] = s3;
    }
  }
  __syncthreads();
  if (col >= d) return;
  for (int ii = warp; ii < ni; ii += kEncWarps) {
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    for (int t = 0; t <= s; ++t) {
      int u = ii + t;  // slot of group (i0 + ii + t) mod n; wraps only when the block holds all n groups
      if (ng == n && u >= n) u -= n;
      const double c = cf[ii * (s + 1) + t];
      const double *gsrc = Gs + u * kEncCols + lane * 4;
      a0 = fma(c, gsrc[0], a0); a1 = fma(c, gsrc[1], a1); a2 = fma(c, gsrc[2], a2); a3 = fma(c, gsrc[3], a3);
    }
    CT *dst = coded + (size_t)(i0 + ii) * d + col;
    if (sizeof(CT) == 8) {
      reinterpret_cast<double2 *>(dst)[0] = make_double2(a0, a1);
      reinterpret_cast<double2 *>(dst)[1] = make_double2(a2, a3);
    } else {
      *reinterpret_cast<float4 *>(dst) = make_float4((float)a0, (float)a1, (float)a2, (float)a3);
    }
  }
}
}  // namespace

namespace {
// Encode for long gradients (dense models, one scratch slot per group): every thread owns 4 columns
// and walks a contiguous chunk of the workers (blockIdx.y), holding a ring of W = S1 + LOOK partial
// gradients in registers exactly as loaded (fp32): S1 = s+1 of them form the worker's window, the
// other LOOK slots are loads in flight for the workers to come, and nothing touches a slot before its
// turn.  The window length is a template parameter, so the inner loops carry no predicates; the
// chunk's coefficients are converted to the coded type once per block into shared memory.  The
// arithmetic is done in the type of the coded gradients (fp32 storage: packed fp32 fused
// multiply-adds, two columns per instruction).  Inside a chunk each partial gradient is read once;
// chunks overlap by s groups, which come from L2.
constexpr int kEncLook = 6;
constexpr int kEncMaxS1 = 12;
constexpr int kEncMaxChunks = kEncodeMaxChunks;

// DEC: the decode rides along.  `avec` is the decoding vector (n weights, zero for workers outside the
// responsive set); each thread also forms sum_i avec[i] * x_i over its chunk of workers from the coded values
// exactly as they are stored, in fp64, and leaves it in gpart[chunk index][d] for `decode_sum_kernel` (or, with a
// single chunk of workers, writes the decoded gradient itself): the coded matrix is not read a second time.
template <typename CT, int S1, bool DEC>
__global__ void __launch_bounds__(128)
encode_window_kernel(const float *__restrict__ ws, long long ld_ws, const double *__restrict__ coef, int n,
                     long long d, int chunk, CT *__restrict__ coded, const double *__restrict__ avec,
                     double *__restrict__ gpart, float *__restrict__ grad) {
  pdl_sync();
  // wide windows keep fewer loads in flight: the ring is what fills the registers (measured at S1 = 11: 3 better than 6)
  constexpr int W = S1 + (S1 >= 8 ? 3 : kEncLook);
  __shared__ CT cs[NGC_MAX_N * S1];
  __shared__ double as[DEC ? NGC_MAX_N : 1];
  const int first = blockIdx.y * chunk;
  const int last = (first + chunk < n) ? first + chunk : n;  // workers first .. last-1
  if (first >= last) return;
  for (int e = threadIdx.x; e < (last - first) * S1; e += 128) cs[e] = (CT)coef[(size_t)first * S1 + e];
  if constexpr (DEC)
    for (int e = threadIdx.x; e < last - first; e += 128) as[e] = avec[first + e];
  __syncthreads();
  const long long col = ((long long)blockIdx.x * 128 + threadIdx.x) * 4;
  if (col >= d) return;
  const int need = last - first + S1 - 1;  // groups first .. first+need-1 (mod n) are read by this chunk
  const float *src = ws + col;
  ulonglong2 win[W];  // each half is a pair of consecutive fp32 columns
  int next = first;   // group that the next free slot receives
  int loaded = 0;
#pragma unroll
  for (int t = 0; t < W; ++t) {
    if (loaded < need) win[t] = __ldg(reinterpret_cast<const ulonglong2 *>(src + (size_t)next * ld_ws));
    ++loaded;
    if (++next == n) next = 0;
  }
  const int store_mode = (d % 4 == 0) ? 4 : (d % 2 == 0) ? 2 : 1;
  const CT *ci = cs;
  CT *dst = coded + (size_t)first * d + col;
  double gacc[4] = {0.0, 0.0, 0.0, 0.0};
  for (int i0 = first; i0 < last; i0 += W) {
#pragma unroll
    for (int t = 0; t < W; ++t) {
      if (i0 + t < last) {
        CT out[4];
        if constexpr (sizeof(CT) == 4) {
          f32x2 a01 = 0ull, a23 = 0ull;
#pragma unroll
          for (int k = 0; k < S1; ++k) {
            const f32x2 cc = pack2(ci[k], ci[k]);
            fma2(a01, cc, win[(t + k) % W].x);
            fma2(a23, cc, win[(t + k) % W].y);
          }
          unpack2(a01, out[0], out[1]);
          unpack2(a23, out[2], out[3]);
        } else {
          out[0] = out[1] = out[2] = out[3] = 0;
#pragma unroll
          for (int k = 0; k < S1; ++k) {
            float g0, g1, g2, g3;
            unpack2(win[(t + k) % W].x, g0, g1);
            unpack2(win[(t + k) % W].y, g2, g3);
            out[0] = fma(ci[k], (CT)g0, out[0]);
            out[1] = fma(ci[k], (CT)g1, out[1]);
            out[2] = fma(ci[k], (CT)g2, out[2]);
            out[3] = fma(ci[k], (CT)g3, out[3]);
          }
        }
        if (store_mode == 4) {
          if constexpr (sizeof(CT) == 8) {
            reinterpret_cast<double2 *>(dst)[0] = make_double2((double)out[0], (double)out[1]);
            reinterpret_cast<double2 *>(dst)[1] = make_double2((double)out[2], (double)out[3]);
          } else {
            *reinterpret_cast<float4 *>(dst) = make_float4((float)out[0], (float)out[1], (float)out[2], (float)out[3]);
          }
        } else if (store_mode == 2) {
          if constexpr (sizeof(CT) == 8) {
            reinterpret_cast<double2 *>(dst)[0] = make_double2((double)out[0], (double)out[1]);
            if (col + 2 < d) reinterpret_cast<double2 *>(dst)[1] = make_double2((double)out[2], (double)out[3]);
          } else {
            reinterpret_cast<float2 *>(dst)[0] = make_float2((float)out[0], (float)out[1]);
            if (col + 2 < d) reinterpret_cast<float2 *>(dst)[1] = make_float2((float)out[2], (float)out[3]);
          }
        } else {
          dst[0] = out[0];
          if (col + 1 < d) dst[1] = out[1];
          if (col + 2 < d) dst[2] = out[2];
          if (col + 3 < d) dst[3] = out[3];
        }
        if constexpr (DEC) {
          const double ai = as[i0 + t - first];
          if (ai != 0.0) {
#pragma unroll
            for (int e = 0; e < 4; ++e) gacc[e] = fma(ai, (double)out[e], gacc[e]);
          }
        }
        ci += S1;
        dst += d;
        // the oldest group is no longer needed; its slot takes the next group of the chunk, if any is left
        if (loaded < need) win[t] = __ldg(reinterpret_cast<const ulonglong2 *>(src + (size_t)next * ld_ws));
        ++loaded;
        if (++next == n) next = 0;
      }
    }
  }
  if constexpr (DEC) {
    if (gridDim.y == 1) {  // a single chunk of workers: this is the decoded gradient
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (col + e < d) grad[col + e] = (float)gacc[e];
    } else {
      double *gp = gpart + (size_t)blockIdx.y * d + col;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (col + e < d) gp[e] = gacc[e];
    }
  }
}

// grad = sum over the worker chunks of the partial decodes, in chunk order.
__global__ void __launch_bounds__(256) decode_sum_kernel(const double *__restrict__ gpart, int chunks, long long d,
                                                         float *__restrict__ grad) {
  pdl_sync();
  const long long col = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= d) return;
  double acc = 0.0;
  for (int c0 = 0; c0 < chunks; c0 += 4) {
    double v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = c0 + i < chunks ? gpart[(size_t)(c0 + i) * d + col] : 0.0;
#pragma unroll
    for (int i = 0; i < 4; ++i) acc += v[i];
  }
  grad[col] = (float)acc;
}

// Plain fallback (very wide windows): one thread per column.
template <typename CT>
__global__ void __launch_bounds__(256)
encode_simple_kernel(const RowSplit split, const float *__restrict__ ws, long long ld_ws,
                     const double *__restrict__ coef, int n, int s, long long d, CT *__restrict__ coded) {
  pdl_sync();
  const long long col = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= d) return;
  for (int i = 0; i < n; ++i) {
    double acc = 0.0;
    for (int t = 0; t <= s; ++t) {
      const int g = (i + t) % n;
      const int c0 = split_owner(split, (long long)g * split.rows_g);
      const int c1 = split_owner(split, (long long)(g + 1) * split.rows_g - 1);
      double gs = 0.0;
      for (int pce = 0; pce <= c1 - c0; ++pce) gs += (double)ws[((size_t)g * split.P + pce) * ld_ws + col];
      acc = fma(coef[(size_t)i * (s + 1) + t], gs, acc);
    }
    coded[(size_t)i * d + col] = (CT)acc;
  }
}

template <typename CT>
using EncodeKernel = void (*)(const float *, long long, const double *, int, long long, int, CT *, const double *, double *,
                              float *);

template <typename CT, bool DEC>
EncodeKernel<CT> encode_window_for(int s1) {
  switch (s1) {
    case 1: return encode_window_kernel<CT, 1, DEC>;
    case 2: return encode_window_kernel<CT, 2, DEC>;
    case 3: return encode_window_kernel<CT, 3, DEC>;
    case 4: return encode_window_kernel<CT, 4, DEC>;
    case 5: return encode_window_kernel<CT, 5, DEC>;
    case 6: return encode_window_kernel<CT, 6, DEC>;
    case 7: return encode_window_kernel<CT, 7, DEC>;
    case 8: return encode_window_kernel<CT, 8, DEC>;
    case 9: return encode_window_kernel<CT, 9, DEC>;
    case 10: return encode_window_kernel<CT, 10, DEC>;
    case 11: return encode_window_kernel<CT, 11, DEC>;
    case 12: return encode_window_kernel<CT, 12, DEC>;
    default: return nullptr;
  }
}

template <typename CT>
cudaError_t encode_long_typed(const RowSplit &split, const float *ws, long long ld_ws, const double *coef, int n, int s,
                              long long d, CT *coded, cudaStream_t stream, const EncodeDecodeArgs *dec) {
  const bool window = split.P == 1 && s + 1 <= kEncMaxS1;
  const bool fuse = window && dec && dec->a && dec->gpart && dec->grad;
  if (dec && dec->fused) *dec->fused = fuse;
  EncodeKernel<CT> kern = !window ? nullptr : (fuse ? encode_window_for<CT, true>(s + 1) : encode_window_for<CT, false>(s + 1));
  if (!kern) {
    launch_k(encode_simple_kernel<CT>, (unsigned)((d + 255) / 256), 256, 0, stream, split, ws, ld_ws, coef, n, s, d, coded);
    return cudaGetLastError();
  }
  // Number of worker chunks: the blocks run in rounds of `capacity` resident blocks, a block's time grows
  // with the groups it reads (chunk + s) plus a fixed part; take the split with the least rounds x time.
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 128, 0);
  if (e != cudaSuccess) return e;
  const long long capacity = (long long)(per_sm > 0 ? per_sm : 1) * device_sm_count();
  const long long col_blocks = (d + 511) / 512;
  int best_chunks = 1;
  long long best_cost = -1;
  for (int chunks = 1; chunks <= n && chunks <= kEncMaxChunks; ++chunks) {
    const int chunk = (n + chunks - 1) / chunks;
    const long long blocks = col_blocks * ((n + chunk - 1) / chunk);
    const long long cost = ((blocks + capacity - 1) / capacity) * (chunk + s + 4);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_chunks = chunks; }
  }
  const int chunk = (n + best_chunks - 1) / best_chunks;
  const dim3 grid((unsigned)col_blocks, (unsigned)((n + chunk - 1) / chunk));
  launch_k(kern, grid, 128, 0, stream, ws, ld_ws, coef, n, d, chunk, coded, fuse ? dec->a : nullptr,
           fuse ? dec->gpart : nullptr, fuse ? dec->grad : nullptr);
  cudaError_t err = cudaGetLastError();
  if (fuse && dec->sum_launches) *dec->sum_launches = grid.y > 1 ? 1 : 0;
  if (err != cudaSuccess || !fuse || grid.y == 1) return err;
  launch_k(decode_sum_kernel, (unsigned)((d + 255) / 256), 256, 0, stream, dec->gpart, (int)grid.y, d, dec->grad);
  return cudaGetLastError();
}
}  // namespace

namespace {
__global__ void __launch_bounds__(256)
sum_slots_kernel(const RowSplit split, const float *__restrict__ ws, long long ld_ws, long long l,
                 float *__restrict__ G_out, long long ld_out) {
  pdl_sync();
  const long long col = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int g = blockIdx.y;
  if (col >= l) return;
  const int c0 = split_owner(split, (long long)g * split.rows_g);
  const int c1 = split_owner(split, (long long)(g + 1) * split.rows_g - 1);
  const float *src = ws + (size_t)g * split.P * ld_ws + col;
  double acc = 0.0;
  for (int pce = 0; pce <= c1 - c0; ++pce) acc += (double)__ldg(src + (size_t)pce * ld_ws);
  G_out[(size_t)g * ld_out + col] = (float)acc;
}
}  // namespace

cudaError_t launch_sum_slots(const RowSplit &split, int n_groups, const float *ws, long long ld_ws, long long l,
                             float *G_out, long long ld_out, cudaStream_t stream) {
  launch_k(sum_slots_kernel, dim3((unsigned)((l + 255) / 256), (unsigned)n_groups), 256, 0, stream, split, ws, ld_ws, l,
           G_out, ld_out);
  return cudaGetLastError();
}

// Encode for the dense models: ws holds [group][slot][ld_ws] fp32, every slot filled, ld_ws a multiple of 4 and >= d.
cudaError_t launch_encode_long(const RowSplit &split, const float *ws, long long ld_ws, const double *d_coef, int n,
                               int s, long long d, void *coded, int coded_dtype, cudaStream_t stream,
                               const EncodeDecodeArgs *dec) {
  if (ld_ws % 4 != 0 || ld_ws < d) return cudaErrorInvalidValue;
  if (coded_dtype == NGC_F64)
    return encode_long_typed<double>(split, ws, ld_ws, d_coef, n, s, d, static_cast<double *>(coded), stream, dec);
  return encode_long_typed<float>(split, ws, ld_ws, d_coef, n, s, d, static_cast<float *>(coded), stream, dec);
}

cudaError_t launch_combine_encode(const RowSplit &split, const float *ws, const double *d_coef, int n, int s, int d,
                                  void *coded, int coded_dtype, cudaStream_t stream) {
  if (d % 4 != 0) return cudaErrorInvalidValue;
  // Few column tiles (small models): 8 workers per block for parallelism, at the price of re-reading
  // (8+s)/8 of the group sums.  Many column tiles: one block takes all n workers and reads everything once.
  const int col_tiles = (d + kEncCols - 1) / kEncCols;
  const int enc_rows = (col_tiles >= 4 * device_sm_count()) ? n : 8;
  dim3 grid(col_tiles, (n + enc_rows - 1) / enc_rows);
  const int held = (enc_rows + s < n) ? enc_rows + s : n;
  const size_t smem = ((size_t)held * kEncCols + (size_t)enc_rows * (s + 1)) * sizeof(double);
  cudaError_t e;
  if (coded_dtype == NGC_F64) {
    e = cudaFuncSetAttribute(combine_encode_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    launch_k(combine_encode_kernel<double>, grid, kEncWarps * 32, smem, stream, split, ws, d_coef, n, s, d,
                                                                          static_cast<double *>(coded), enc_rows);
  } else {
    e = cudaFuncSetAttribute(combine_encode_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    launch_k(combine_encode_kernel<float>, grid, kEncWarps * 32, smem, stream, split, ws, d_coef, n, s, d,
                                                                         static_cast<float *>(coded), enc_rows);
  }
  return cudaGetLastError();
}

}  // namespace ngc
