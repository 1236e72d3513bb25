// Dense-contraction partial gradients (Section II-C: g_j = sum over the rows of partition j of the
// per-sample loss gradient) on the tensor cores.
//   softmax regression:  forward   Z = X_j W,  R = softmax(Z) - onehot(y_j)      (epilogue fused, R bf16)
//                        backward  g_j = X_j^T R                                 (fp32, written once)
//   784-512-10 style MLP: forward  pre = [X_j 1] [W1; b1], h = relu(pre), z = h W2 + b2,
//                                  delta2 = softmax(z) - onehot, delta1 = (delta2 W2^T) * (pre > 0)
//                        backward  [dW1; db1] = [X_j 1]^T delta1,  [dW2; db2] = [h 1]^T delta2
// All contractions run on tcgen05 with accumulators in tensor memory.  Operands reach shared memory through
// TMA tensor maps with the 128-byte swizzle; the forward reads X and W^T K-major, the backward reads
// the very same X and R row-major as M/N-major operands, so no transposed copy of the data exists.
// Warp roles per CTA: warp 0 TMA producer, warp 1 MMA issuer (+ tensor-memory owner), warps 2-5
// epilogue (one accumulator row per thread).  Two 256-column accumulators let the epilogue of one
// tile overlap the contraction of the next.
#include "ngc_device.h"
#include "ngc_tc.cuh"

namespace ngc {

namespace {

using namespace tc;

constexpr int kStages = 4;
constexpr int kABytes = 128 * 64 * 2;  // 16 KB: 128 x 64 bf16
constexpr int kBBytes = 256 * 64 * 2;  // 32 KB: 256 x 64 bf16
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kTcThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kSmemTc = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;

struct TcParams {
  int k;       // partitions
  int rows;    // rows per partition
  int d;       // features
  int C;       // classes (multiple of 16, <= 256)
  int tiles_per_part;
  int num_tiles;
  int num_k;   // K chunks of 64
  const int *y;
  __nv_bfloat16 *R;   // [k][rows][C]
  int *status;
};

// D[M x N] = A^T B per batch, A stored [batch][K][M] and B stored [batch][K][N_total] (both row-major bf16,
// read as M/N-major operands).  Tile = (batch j, 128 rows of M, 256 columns of N_total).
struct TnParams {
  int batch, m_tiles, n_tiles, num_tiles;
  int num_k;      // K chunks of 64
  int N;          // columns per MMA (multiple of 16, <= 256)
  int nbox;       // 64-column boxes of B per stage
  int m_store;    // rows of D that exist
  int n_store;    // columns of a tile's D that are stored
  float *out;     // D(j, m, nt*256 + c) -> out[j * out_batch + m * out_ld + nt * 256 + c]
  size_t out_batch;
  int out_ld;
  int *status;
};

struct Smem {
  unsigned char *tiles;
  uint32_t full[kStages], empty[kStages], tfull[2], tempty[2];
  uint32_t *tmem_slot;
  volatile int *abort_flag;
};

__device__ __forceinline__ Smem carve(unsigned char *raw) {
  Smem s;
  const uint32_t base = smem_u32(raw);
  s.tiles = raw + ((1024u - (base & 1023u)) & 1023u);
  uint64_t *bars = reinterpret_cast<uint64_t *>(s.tiles + kStages * kStageBytes);
  for (int i = 0; i < kStages; ++i) {
    s.full[i] = smem_u32(&bars[i]);
    s.empty[i] = smem_u32(&bars[kStages + i]);
  }
  s.tfull[0] = smem_u32(&bars[2 * kStages]);
  s.tfull[1] = smem_u32(&bars[2 * kStages + 1]);
  s.tempty[0] = smem_u32(&bars[2 * kStages + 2]);
  s.tempty[1] = smem_u32(&bars[2 * kStages + 3]);
  s.tmem_slot = reinterpret_cast<uint32_t *>(&bars[2 * kStages + 4]);
  s.abort_flag = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
  return s;
}

// Common prologue: barriers, tensor memory.  Returns the tensor-memory base address.
__device__ __forceinline__ uint32_t prologue(const Smem &s, int warp) {
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(s.full[i], 1);
      mbar_init(s.empty[i], 1);
    }
    mbar_init(s.tfull[0], 1);
    mbar_init(s.tfull[1], 1);
    mbar_init(s.tempty[0], 128);
    mbar_init(s.tempty[1], 128);
    *s.abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(s.tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  return *s.tmem_slot;
}

__device__ __forceinline__ void epilogue_teardown(const Smem &s, int warp, uint32_t tmem_base, bool failed,
                                                  int *status) {
  if (failed) {
    *s.abort_flag = 1;
    atomicExch(status, 1);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------------------------
// W (fp32, [d][C]) -> W^T (bf16, [C][ld]): the K-major B operand of a forward contraction.  With a
// bias vector, column d of W^T holds it (the data matrix then carries a matching column of ones);
// columns beyond are zero.
// ------------------------------------------------------------------------------------------------
__global__ void transpose_to_bf16_kernel(const float *__restrict__ W, const float *__restrict__ bias,
                                         __nv_bfloat16 *__restrict__ Wt, int d, int C, int ld) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, d0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int dd = d0 + r, c = c0 + threadIdx.x;
    float v = 0.f;
    if (c < C) {
      if (dd < d) v = W[(size_t)dd * C + c];
      else if (dd == d && bias) v = bias[c];
    }
    tile[r][threadIdx.x] = v;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int c = c0 + r, dd = d0 + threadIdx.x;
    if (c < C && dd < ld) Wt[(size_t)c * ld + dd] = __float2bfloat16_rn(tile[threadIdx.x][r]);
  }
}

// X (fp32, [rows_total][d]) -> bf16 [rows_total][ld] with a column of ones at index d and zeros after
// it: the ones column turns the bias of the first layer, and the bias gradient, into one more row of
// the weight contraction.  One thread per 8 output columns.
__global__ void convert_x_kernel(const float *__restrict__ X, __nv_bfloat16 *__restrict__ Xb, long long rows_total,
                                 int d, int ld) {
  const int groups = ld / 8;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows_total * groups) return;
  const long long row = idx / groups;
  const int c0 = (int)(idx % groups) * 8;
  float v[8];
  if (c0 + 8 <= d) {
    const float4 a = __ldg(reinterpret_cast<const float4 *>(X + row * d + c0));
    const float4 b = __ldg(reinterpret_cast<const float4 *>(X + row * d + c0 + 4));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int c = c0 + i;
      v[i] = c < d ? X[row * d + c] : (c == d ? 1.f : 0.f);
    }
  }
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<const uint32_t *>(&b2);
  }
  *reinterpret_cast<uint4 *>(Xb + row * ld + c0) = make_uint4(w[0], w[1], w[2], w[3]);
}

// ------------------------------------------------------------------------------------------------
// Forward: tile = (partition j, block of 128 rows).  D[128 x C] = X_tile[128 x d] * W[d x C].
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTcThreads, 1)
softmax_fwd_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const Smem s = carve(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_base = prologue(s, warp);
  bool failed = false;

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        const int j = tile / p.tiles_per_part, rb = tile % p.tiles_per_part;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.empty[st], ph ^ 1u)) { failed = true; break; }
          mbar_expect_tx(s.full[st], kStageBytes);
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          tma_load_3d(a, &tmX, kc * 64, rb * 128, j, s.full[st]);
          tma_load_2d(a + kABytes, &tmW, kc * 64, 0, s.full[st]);
          if (++st == kStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(128, p.C, 0, 0);
      int st = 0, buf = 0;
      uint32_t ph = 0, aph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        if (!mbar_wait(s.tempty[buf], aph ^ 1u)) { failed = true; break; }
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)buf * 256u;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.full[st], ph)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          const uint64_t ad = smem_desc_sw128(a, 16, 1024), bd = smem_desc_sw128(a + kABytes, 16, 1024);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)  // 16 bf16 = 32 bytes along K per instruction
            mma_bf16(acc, ad + (uint64_t)(k4 * 2), bd + (uint64_t)(k4 * 2), idesc, (kc | k4) != 0);
          mma_commit(s.empty[st]);
          if (++st == kStages) { st = 0; ph ^= 1u; }
        }
        if (failed) break;
        mma_commit(s.tfull[buf]);
        buf ^= 1;
        if (buf == 0) aph ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;  // the 32-lane quadrant of tensor memory this warp may read
    int buf = 0;
    uint32_t aph = 0;
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int j = tile / p.tiles_per_part, rb = tile % p.tiles_per_part;
      if (!mbar_wait(s.tfull[buf], aph)) { failed = true; break; }
      tc_fence_after();
      const int row = rb * 128 + q * 32 + lane;
      const bool valid = row < p.rows;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 256u;
      const int label = valid ? p.y[(size_t)j * p.rows + row] : -1;
      float v[32];
      float mx = -INFINITY;
      for (int c0 = 0; c0 < p.C; c0 += 32) {
        tmem_ld32(taddr + c0, v);
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (c0 + i < p.C) mx = fmaxf(mx, v[i]);
      }
      float sum = 0.f;
      for (int c0 = 0; c0 < p.C; c0 += 32) {
        tmem_ld32(taddr + c0, v);
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (c0 + i < p.C) sum += __expf(v[i] - mx);
      }
      const float inv = 1.f / sum;
      __nv_bfloat16 *dst = p.R + ((size_t)j * p.rows + (valid ? row : 0)) * p.C;
      for (int c0 = 0; c0 < p.C; c0 += 32) {
        tmem_ld32(taddr + c0, v);
#pragma unroll
        for (int g8 = 0; g8 < 4; ++g8) {
          uint32_t w[4];
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            const int c = c0 + g8 * 8 + h * 2;
            const float r0 = __expf(v[g8 * 8 + h * 2] - mx) * inv - (c == label ? 1.f : 0.f);
            const float r1 = __expf(v[g8 * 8 + h * 2 + 1] - mx) * inv - (c + 1 == label ? 1.f : 0.f);
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(r0, r1);
            w[h] = *reinterpret_cast<const uint32_t *>(&b2);
          }
          if (valid && c0 + g8 * 8 < p.C) *reinterpret_cast<uint4 *>(dst + c0 + g8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      tc_fence_before();
      mbar_arrive(s.tempty[buf]);
      buf ^= 1;
      if (buf == 0) aph ^= 1u;
    }
  }
  epilogue_teardown(s, warp, tmem_base, failed, p.status);
}

// ------------------------------------------------------------------------------------------------
// Backward contractions: D = A^T B with K = the partition's rows (see TnParams).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTcThreads, 1)
tn_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TnParams p) {
  extern __shared__ unsigned char smem_raw[];
  const Smem s = carve(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_base = prologue(s, warp);
  bool failed = false;

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      const uint32_t tx = (uint32_t)(2 + p.nbox) * 8192u;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        const int nt = tile % p.n_tiles, mt = (tile / p.n_tiles) % p.m_tiles, j = tile / (p.n_tiles * p.m_tiles);
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.empty[st], ph ^ 1u)) { failed = true; break; }
          mbar_expect_tx(s.full[st], tx);
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          tma_load_3d(a, &tmA, mt * 128, kc * 64, j, s.full[st]);
          tma_load_3d(a + 8192, &tmA, mt * 128 + 64, kc * 64, j, s.full[st]);
          for (int nb = 0; nb < p.nbox; ++nb)
            tma_load_3d(a + kABytes + nb * 8192, &tmB, nt * 256 + nb * 64, kc * 64, j, s.full[st]);
          if (++st == kStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(128, p.N, 1, 1);
      int st = 0, buf = 0;
      uint32_t ph = 0, aph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        if (!mbar_wait(s.tempty[buf], aph ^ 1u)) { failed = true; break; }
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)buf * 256u;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.full[st], ph)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          // M/N-major: 64-element boxes 8192 B apart, 8-row K groups 1024 B apart
          const uint64_t ad = smem_desc_sw128(a, 8192, 1024), bd = smem_desc_sw128(a + kABytes, 8192, 1024);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)  // 16 rows of K = 2048 bytes per instruction
            mma_bf16(acc, ad + (uint64_t)(k4 * 128), bd + (uint64_t)(k4 * 128), idesc, (kc | k4) != 0);
          mma_commit(s.empty[st]);
          if (++st == kStages) { st = 0; ph ^= 1u; }
        }
        if (failed) break;
        mma_commit(s.tfull[buf]);
        buf ^= 1;
        if (buf == 0) aph ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;
    int buf = 0;
    uint32_t aph = 0;
    const bool vec = (p.out_ld % 4 == 0) && (p.n_store % 4 == 0) && (p.out_batch % 4 == 0);
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int nt = tile % p.n_tiles, mt = (tile / p.n_tiles) % p.m_tiles, j = tile / (p.n_tiles * p.m_tiles);
      if (!mbar_wait(s.tfull[buf], aph)) { failed = true; break; }
      tc_fence_after();
      const int m = mt * 128 + q * 32 + lane;
      const bool valid = m < p.m_store;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 256u;
      float *dst = p.out + (size_t)j * p.out_batch + (size_t)(valid ? m : 0) * p.out_ld + (size_t)nt * 256;
      float v[32];
      for (int c0 = 0; c0 < p.n_store; c0 += 32) {
        tmem_ld32(taddr + c0, v);
        if (valid) {
          if (vec) {
#pragma unroll
            for (int g4 = 0; g4 < 8; ++g4)
              if (c0 + g4 * 4 < p.n_store)
                *reinterpret_cast<float4 *>(dst + c0 + g4 * 4) = make_float4(v[g4 * 4], v[g4 * 4 + 1], v[g4 * 4 + 2], v[g4 * 4 + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + i < p.n_store) dst[c0 + i] = v[i];
          }
        }
      }
      tc_fence_before();
      mbar_arrive(s.tempty[buf]);
      buf ^= 1;
      if (buf == 0) aph ^= 1u;
    }
  }
  epilogue_teardown(s, warp, tmem_base, failed, p.status);
}

// ------------------------------------------------------------------------------------------------
// MLP forward: tile = (partition j, block of 128 rows).  pre[128 x hidden] = [X 1][W1; b1] in tensor
// memory (up to two 256-column accumulators), then on the CUDA cores, one thread per (row, half of the
// hidden units): h = relu(pre), z = h W2 + b2, delta2 = softmax(z) - onehot(y),
// delta1 = (delta2 W2^T) * (pre > 0).  Stored for the backward contractions: H = [h 1] and delta1 as
// bf16 row-major, delta2 as bf16 rows of 64 (16 used).
// ------------------------------------------------------------------------------------------------
constexpr int kMlpStages = 2;
constexpr int kMlpBBytes = 512 * 64 * 2;  // 64 KB: up to 512 hidden units x 64 bf16
constexpr int kMlpStageBytes = kABytes + kMlpBBytes;
constexpr int kMlpThreads = 320;          // producer, MMA, 8 epilogue warps

struct MlpParams {
  int k, rows, d, hidden, C;
  int hpad;      // row stride of H = hidden + 1 rounded up to 8
  int tiles_per_part, num_tiles, num_k;
  const int *y;
  const float *W2;   // [hidden][C]
  const float *b2;   // [C]
  __nv_bfloat16 *H;  // [k][rows][hpad]
  __nv_bfloat16 *D1; // [k][rows][hidden]
  __nv_bfloat16 *D2; // [k][rows][64]
  int *status;
};

template <int CPAD>
__global__ void __launch_bounds__(kMlpThreads, 1)
mlp_fwd_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const MlpParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char *tiles = smem_raw + ((1024u - (base & 1023u)) & 1023u);
  uint64_t *bars = reinterpret_cast<uint64_t *>(tiles + kMlpStages * kMlpStageBytes);
  uint32_t full[kMlpStages], empty[kMlpStages];
#pragma unroll
  for (int i = 0; i < kMlpStages; ++i) {
    full[i] = smem_u32(&bars[i]);
    empty[i] = smem_u32(&bars[kMlpStages + i]);
  }
  const uint32_t tfull = smem_u32(&bars[2 * kMlpStages]), tempty = smem_u32(&bars[2 * kMlpStages + 1]);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(&bars[2 * kMlpStages + 2]);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *W2s = reinterpret_cast<float *>(tiles + kMlpStages * kMlpStageBytes + 128);  // [hidden][CPAD]
  float *b2s = W2s + 512 * CPAD;                                                      // [CPAD]
  float *zpart = b2s + 16;                                                            // [2][128][CPAD]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMlpStages; ++i) {
      mbar_init(full[i], 1);
      mbar_init(empty[i], 1);
    }
    mbar_init(tfull, 1);
    mbar_init(tempty, 256);
    *abort_flag = 0;
    mbar_fence_init();
  }
  for (int e = threadIdx.x; e < p.hidden * CPAD; e += kMlpThreads) {
    const int hc = e / CPAD, c = e % CPAD;
    W2s[e] = c < p.C ? p.W2[(size_t)hc * p.C + c] : 0.f;
  }
  if (threadIdx.x < CPAD) b2s[threadIdx.x] = threadIdx.x < p.C ? p.b2[threadIdx.x] : 0.f;
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;
  const int n_halves = (p.hidden + 255) / 256;

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      const uint32_t tx = (uint32_t)kABytes + (uint32_t)n_halves * 32768u;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        const int j = tile / p.tiles_per_part, rb = tile % p.tiles_per_part;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(empty[st], ph ^ 1u)) { failed = true; break; }
          mbar_expect_tx(full[st], tx);
          const uint32_t a = smem_u32(tiles + st * kMlpStageBytes);
          tma_load_3d(a, &tmX, kc * 64, rb * 128, j, full[st]);
          for (int h = 0; h < n_halves; ++h) tma_load_2d(a + kABytes + h * 32768, &tmW, kc * 64, h * 256, full[st]);
          if (++st == kMlpStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0, aph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        if (!mbar_wait(tempty, aph ^ 1u)) { failed = true; break; }
        tc_fence_after();
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(full[st], ph)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(tiles + st * kMlpStageBytes);
          const uint64_t ad = smem_desc_sw128(a, 16, 1024);
          for (int h = 0; h < n_halves; ++h) {
            const int nh = min(256, p.hidden - h * 256);
            const uint32_t idesc = instr_desc_bf16(128, nh, 0, 0);
            const uint64_t bd = smem_desc_sw128(a + kABytes + h * 32768, 16, 1024);
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4)
              mma_bf16(tmem_base + (uint32_t)h * 256u, ad + (uint64_t)(k4 * 2), bd + (uint64_t)(k4 * 2), idesc,
                       (kc | k4) != 0);
          }
          mma_commit(empty[st]);
          if (++st == kMlpStages) { st = 0; ph ^= 1u; }
        }
        if (failed) break;
        mma_commit(tfull);
        aph ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;           // tensor-memory quadrant of this warp
    const int hf = (warp - 2) >> 2;   // which 256 hidden units
    const int rt = q * 32 + lane;     // row within the tile
    const int h_begin = hf * 256, h_count = max(0, min(256, p.hidden - h_begin));
    uint32_t aph = 0;
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int j = tile / p.tiles_per_part, rb = tile % p.tiles_per_part;
      if (!mbar_wait(tfull, aph)) { failed = true; break; }
      tc_fence_after();
      const int row = rb * 128 + rt;
      const bool valid = row < p.rows;
      const size_t grow = (size_t)j * p.rows + (valid ? row : 0);
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)h_begin;
      const int label = valid ? p.y[grow] : -1;
      float v[32];
      float z[CPAD];
#pragma unroll
      for (int c = 0; c < CPAD; ++c) z[c] = 0.f;
      for (int c0 = 0; c0 < h_count; c0 += 32) {
        tmem_ld32(taddr + c0, v);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (c0 + i < h_count) {
            const float h = fmaxf(v[i], 0.f);
            const float4 *w2 = reinterpret_cast<const float4 *>(W2s + (size_t)(h_begin + c0 + i) * CPAD);
#pragma unroll
            for (int c4 = 0; c4 < CPAD / 4; ++c4) {
              const float4 ww = w2[c4];
              z[c4 * 4] = fmaf(h, ww.x, z[c4 * 4]);
              z[c4 * 4 + 1] = fmaf(h, ww.y, z[c4 * 4 + 1]);
              z[c4 * 4 + 2] = fmaf(h, ww.z, z[c4 * 4 + 2]);
              z[c4 * 4 + 3] = fmaf(h, ww.w, z[c4 * 4 + 3]);
            }
          }
        }
      }
#pragma unroll
      for (int c = 0; c < CPAD; ++c) zpart[(hf * 128 + rt) * CPAD + c] = z[c];
      asm volatile("bar.sync 1, 256;" ::: "memory");
      float dl[CPAD];
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < CPAD; ++c) {
        z[c] = zpart[rt * CPAD + c] + zpart[(128 + rt) * CPAD + c] + b2s[c];
        if (c < p.C) mx = fmaxf(mx, z[c]);
      }
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < CPAD; ++c) {
        dl[c] = c < p.C ? __expf(z[c] - mx) : 0.f;
        sum += dl[c];
      }
      const float inv = 1.f / sum;
#pragma unroll
      for (int c = 0; c < CPAD; ++c) dl[c] = c < p.C ? dl[c] * inv - (c == label ? 1.f : 0.f) : 0.f;
      if (hf == 0 && valid) {
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float lo = 2 * i < CPAD ? dl[2 * i < CPAD ? 2 * i : 0] : 0.f;
          const float hi = 2 * i + 1 < CPAD ? dl[2 * i + 1 < CPAD ? 2 * i + 1 : 0] : 0.f;
          const __nv_bfloat162 b2v = __floats2bfloat162_rn(lo, hi);
          w[i] = *reinterpret_cast<const uint32_t *>(&b2v);
        }
        uint4 *d2 = reinterpret_cast<uint4 *>(p.D2 + grow * 64);
        d2[0] = make_uint4(w[0], w[1], w[2], w[3]);
        d2[1] = make_uint4(w[4], w[5], w[6], w[7]);
        // column of ones (and padding) behind the hidden activations
        *reinterpret_cast<uint4 *>(p.H + grow * p.hpad + p.hidden) = make_uint4(0x00003f80u, 0u, 0u, 0u);
      }
      __nv_bfloat16 *hrow = p.H + grow * p.hpad + h_begin;
      __nv_bfloat16 *drow = p.D1 + grow * p.hidden + h_begin;
      for (int c0 = 0; c0 < h_count; c0 += 32) {
        tmem_ld32(taddr + c0, v);
#pragma unroll
        for (int g8 = 0; g8 < 4; ++g8) {
          uint32_t hw[4], dw[4];
#pragma unroll
          for (int hh = 0; hh < 4; ++hh) {
            float hv[2], dv[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              const int i = g8 * 8 + hh * 2 + u;
              const float pre = v[i];
              const bool act = pre > 0.f && (c0 + i < h_count);
              const int hc = min(h_begin + c0 + i, p.hidden - 1);
              const float4 *w2 = reinterpret_cast<const float4 *>(W2s + (size_t)hc * CPAD);
              float acc = 0.f;
#pragma unroll
              for (int c4 = 0; c4 < CPAD / 4; ++c4) {
                const float4 ww = w2[c4];
                acc = fmaf(dl[c4 * 4], ww.x, acc);
                acc = fmaf(dl[c4 * 4 + 1], ww.y, acc);
                acc = fmaf(dl[c4 * 4 + 2], ww.z, acc);
                acc = fmaf(dl[c4 * 4 + 3], ww.w, acc);
              }
              hv[u] = act ? pre : 0.f;
              dv[u] = act ? acc : 0.f;
            }
            const __nv_bfloat162 hb = __floats2bfloat162_rn(hv[0], hv[1]);
            const __nv_bfloat162 db = __floats2bfloat162_rn(dv[0], dv[1]);
            hw[hh] = *reinterpret_cast<const uint32_t *>(&hb);
            dw[hh] = *reinterpret_cast<const uint32_t *>(&db);
          }
          if (valid && c0 + g8 * 8 < h_count) {
            *reinterpret_cast<uint4 *>(hrow + c0 + g8 * 8) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
            *reinterpret_cast<uint4 *>(drow + c0 + g8 * 8) = make_uint4(dw[0], dw[1], dw[2], dw[3]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(tempty);
      aph ^= 1u;
    }
  }
  if (failed) {
    *abort_flag = 1;
    atomicExch(p.status, 1);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------------------------
// Host side: tensor maps
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 tensor, innermost dimension first; 128-byte swizzle; out-of-range elements read as zero.
bool make_map(CUtensorMap *m, const void *base, int rank, const uint64_t *dims, const uint32_t *box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[3], gstr[2];
  cuuint32_t bx[3], es[3];
  uint64_t stride = 2;
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    stride *= dims[i];
    if (i < rank - 1) gstr[i] = stride;
  }
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), gdim, gstr, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t softmax_scratch_bytes(int k, int rows, int d, int C) {
  const size_t wt = ((size_t)C * d * 2 + 255) / 256 * 256;
  const size_t r = ((size_t)k * rows * C * 2 + 255) / 256 * 256;
  const size_t g = (size_t)k * d * C * 4;
  return wt + r + g;
}

cudaError_t launch_softmax_grad(int k, int rows, int d, int C, const void *X, const int *y, const float *W,
                                unsigned char *scratch, float **G_out, int *status, int sms, cudaStream_t stream) {
  if (C % 16 != 0 || C < 16 || C > 256 || d % 8 != 0 || d < 8) return cudaErrorInvalidValue;
  const size_t wt_bytes = ((size_t)C * d * 2 + 255) / 256 * 256;
  const size_t r_bytes = ((size_t)k * rows * C * 2 + 255) / 256 * 256;
  __nv_bfloat16 *Wt = reinterpret_cast<__nv_bfloat16 *>(scratch);
  __nv_bfloat16 *R = reinterpret_cast<__nv_bfloat16 *>(scratch + wt_bytes);
  float *G = reinterpret_cast<float *>(scratch + wt_bytes + r_bytes);
  *G_out = G;

  CUtensorMap tmXa, tmXb, tmW, tmR;
  const uint64_t xdims[3] = {(uint64_t)d, (uint64_t)rows, (uint64_t)k};
  const uint32_t xbox_a[3] = {64, 128, 1}, xbox_b[3] = {64, 64, 1};
  const uint64_t wdims[2] = {(uint64_t)d, (uint64_t)C};
  const uint32_t wbox[2] = {64, 256};
  const uint64_t rdims[3] = {(uint64_t)C, (uint64_t)rows, (uint64_t)k};
  const uint32_t rbox[3] = {64, 64, 1};
  if (!make_map(&tmXa, X, 3, xdims, xbox_a) || !make_map(&tmXb, X, 3, xdims, xbox_b) ||
      !make_map(&tmW, Wt, 2, wdims, wbox) || !make_map(&tmR, R, 3, rdims, rbox))
    return cudaErrorInvalidValue;

  dim3 tb(32, 8), tg((C + 31) / 32, (d + 31) / 32);
  transpose_to_bf16_kernel<<<tg, tb, 0, stream>>>(W, nullptr, Wt, d, C, d);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  TcParams p;
  p.k = k; p.rows = rows; p.d = d; p.C = C;
  p.y = y; p.R = R; p.status = status;

  e = cudaFuncSetAttribute(softmax_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(tn_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc);
  if (e != cudaSuccess) return e;

  p.tiles_per_part = (rows + 127) / 128;
  p.num_tiles = k * p.tiles_per_part;
  p.num_k = (d + 63) / 64;
  softmax_fwd_kernel<<<p.num_tiles < sms ? p.num_tiles : sms, kTcThreads, kSmemTc, stream>>>(tmXa, tmW, p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  TnParams t;
  t.batch = k; t.m_tiles = (d + 127) / 128; t.n_tiles = 1; t.num_tiles = k * t.m_tiles;
  t.num_k = (rows + 63) / 64;
  t.N = C; t.nbox = (C + 63) / 64;
  t.m_store = d; t.n_store = C;
  t.out = G; t.out_batch = (size_t)d * C; t.out_ld = C;
  t.status = status;
  tn_gemm_kernel<<<t.num_tiles < sms ? t.num_tiles : sms, kTcThreads, kSmemTc, stream>>>(tmXb, tmR, t);
  return cudaGetLastError();
}


namespace {
inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }
}  // namespace

size_t mlp_scratch_bytes(int k, int rows, int d, int hidden, int C) {
  const size_t dpad = (size_t)(d + 1 + 7) / 8 * 8, hpad = (size_t)(hidden + 1 + 7) / 8 * 8;
  const size_t l = (size_t)d * hidden + hidden + (size_t)hidden * C + C, lpad = (l + 3) / 4 * 4;
  const size_t kr = (size_t)k * rows;
  return up256(kr * dpad * 2) + up256((size_t)hidden * dpad * 2) + up256(kr * hpad * 2) + up256(kr * hidden * 2) +
         up256(kr * 64 * 2) + up256((size_t)k * lpad * 4);
}

cudaError_t launch_mlp_grad(int k, int rows, int d, int hidden, int C, const float *X, const int *y, const float *theta,
                            unsigned char *scratch, float **G_out, long long *G_ld, int *status, int sms,
                            cudaStream_t stream) {
  if (d % 8 != 0 || hidden % 16 != 0 || hidden < 16 || hidden > 512 || (hidden > 256 && hidden % 256 != 0) || C < 1 ||
      C > 16)
    return cudaErrorInvalidValue;
  const int dpad = (d + 1 + 7) / 8 * 8, hpad = (hidden + 1 + 7) / 8 * 8;
  const size_t l = (size_t)d * hidden + hidden + (size_t)hidden * C + C, lpad = (l + 3) / 4 * 4;
  const size_t kr = (size_t)k * rows;
  unsigned char *ptr = scratch;
  __nv_bfloat16 *Xb = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * dpad * 2);
  __nv_bfloat16 *W1t = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256((size_t)hidden * dpad * 2);
  __nv_bfloat16 *H = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * hpad * 2);
  __nv_bfloat16 *D1 = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * hidden * 2);
  __nv_bfloat16 *D2 = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * 64 * 2);
  float *G = reinterpret_cast<float *>(ptr);
  *G_out = G;
  *G_ld = (long long)lpad;
  const float *W1 = theta, *b1 = theta + (size_t)d * hidden, *W2 = b1 + hidden, *b2 = W2 + (size_t)hidden * C;

  CUtensorMap tmXa, tmXb, tmW, tmH, tmD1, tmD2;
  const uint64_t xdims[3] = {(uint64_t)dpad, (uint64_t)rows, (uint64_t)k};
  const uint32_t box_a[3] = {64, 128, 1}, box_b[3] = {64, 64, 1};
  const uint64_t wdims[2] = {(uint64_t)dpad, (uint64_t)hidden};
  const uint32_t wbox[2] = {64, 256};
  const uint64_t hdims[3] = {(uint64_t)hpad, (uint64_t)rows, (uint64_t)k};
  const uint64_t d1dims[3] = {(uint64_t)hidden, (uint64_t)rows, (uint64_t)k};
  const uint64_t d2dims[3] = {64, (uint64_t)rows, (uint64_t)k};
  if (!make_map(&tmXa, Xb, 3, xdims, box_a) || !make_map(&tmXb, Xb, 3, xdims, box_b) ||
      !make_map(&tmW, W1t, 2, wdims, wbox) || !make_map(&tmH, H, 3, hdims, box_b) ||
      !make_map(&tmD1, D1, 3, d1dims, box_b) || !make_map(&tmD2, D2, 3, d2dims, box_b))
    return cudaErrorInvalidValue;

  const long long groups = (long long)kr * (dpad / 8);
  convert_x_kernel<<<(unsigned)((groups + 255) / 256), 256, 0, stream>>>(X, Xb, (long long)kr, d, dpad);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 tb(32, 8), tg((hidden + 31) / 32, (dpad + 31) / 32);
  transpose_to_bf16_kernel<<<tg, tb, 0, stream>>>(W1, b1, W1t, d, hidden, dpad);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;

  MlpParams p;
  p.k = k; p.rows = rows; p.d = d; p.hidden = hidden; p.C = C; p.hpad = hpad;
  p.tiles_per_part = (rows + 127) / 128;
  p.num_tiles = k * p.tiles_per_part;
  p.num_k = (dpad + 63) / 64;
  p.y = y; p.W2 = W2; p.b2 = b2; p.H = H; p.D1 = D1; p.D2 = D2; p.status = status;
  const int cpad = (C + 3) / 4 * 4;
  const int smem = kMlpStages * kMlpStageBytes + 1024 + 128 + (512 * cpad + 16 + 2 * 128 * cpad) * 4;
  const int grid = p.num_tiles < sms ? p.num_tiles : sms;
#define NGC_LAUNCH_MLP(CP)                                                                                   \
  do {                                                                                                       \
    e = cudaFuncSetAttribute(mlp_fwd_kernel<CP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);         \
    if (e != cudaSuccess) return e;                                                                          \
    mlp_fwd_kernel<CP><<<grid, kMlpThreads, smem, stream>>>(tmXa, tmW, p);                                    \
  } while (0)
  if (cpad == 4) NGC_LAUNCH_MLP(4);
  else if (cpad == 8) NGC_LAUNCH_MLP(8);
  else if (cpad == 12) NGC_LAUNCH_MLP(12);
  else NGC_LAUNCH_MLP(16);
#undef NGC_LAUNCH_MLP
  if ((e = cudaGetLastError()) != cudaSuccess) return e;

  e = cudaFuncSetAttribute(tn_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc);
  if (e != cudaSuccess) return e;
  TnParams t;
  t.batch = k; t.status = status; t.num_k = (rows + 63) / 64;
  // [dW1; db1] = [X 1]^T delta1
  t.m_tiles = (d + 1 + 127) / 128; t.n_tiles = (hidden + 255) / 256; t.num_tiles = k * t.m_tiles * t.n_tiles;
  t.N = hidden < 256 ? hidden : 256; t.nbox = (t.N + 63) / 64;
  t.m_store = d + 1; t.n_store = t.N;
  t.out = G; t.out_batch = lpad; t.out_ld = hidden;
  tn_gemm_kernel<<<t.num_tiles < sms ? t.num_tiles : sms, kTcThreads, kSmemTc, stream>>>(tmXb, tmD1, t);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // [dW2; db2] = [h 1]^T delta2
  t.m_tiles = (hidden + 1 + 127) / 128; t.n_tiles = 1; t.num_tiles = k * t.m_tiles;
  t.N = 16; t.nbox = 1;
  t.m_store = hidden + 1; t.n_store = C;
  t.out = G + (size_t)d * hidden + hidden; t.out_batch = lpad; t.out_ld = C;
  tn_gemm_kernel<<<t.num_tiles < sms ? t.num_tiles : sms, kTcThreads, kSmemTc, stream>>>(tmH, tmD2, t);
  return cudaGetLastError();
}

}  // namespace ngc
