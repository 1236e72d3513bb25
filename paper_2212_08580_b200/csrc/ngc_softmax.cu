// Softmax-regression partial gradients (Section II-C: g_j = sum over the rows of partition j of the
// per-sample loss gradient) as two tensor-core contractions per partition:
//     forward   Z = X_j W,  R = softmax(Z) - onehot(y_j)          (epilogue fused, R stored as bf16)
//     backward  g_j = X_j^T R                                     (fp32, written once)
// Both run on tcgen05 with accumulators in tensor memory.  Operands reach shared memory through
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
  float *G;           // [k][d*C]
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
// W (fp32, [d][C]) -> W^T (bf16, [C][d]): the K-major B operand of the forward contraction.
// ------------------------------------------------------------------------------------------------
__global__ void transpose_to_bf16_kernel(const float *__restrict__ W, __nv_bfloat16 *__restrict__ Wt, int d, int C) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, d0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int dd = d0 + r, c = c0 + threadIdx.x;
    tile[r][threadIdx.x] = (dd < d && c < C) ? W[(size_t)dd * C + c] : 0.f;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int c = c0 + r, dd = d0 + threadIdx.x;
    if (c < C && dd < d) Wt[(size_t)c * d + dd] = __float2bfloat16_rn(tile[threadIdx.x][r]);
  }
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
// Backward: tile = (partition j, block of 128 features).  D[128 x C] = X_j[:, block]^T * R_j, K = rows.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTcThreads, 1)
softmax_bwd_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR, const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const Smem s = carve(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_base = prologue(s, warp);
  bool failed = false;
  const int nbox = (p.C + 63) / 64;  // 64-class boxes of R per stage

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      const uint32_t tx = (uint32_t)(2 + nbox) * 8192u;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        const int j = tile / p.tiles_per_part, mt = tile % p.tiles_per_part;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.empty[st], ph ^ 1u)) { failed = true; break; }
          mbar_expect_tx(s.full[st], tx);
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          tma_load_3d(a, &tmX, mt * 128, kc * 64, j, s.full[st]);
          tma_load_3d(a + 8192, &tmX, mt * 128 + 64, kc * 64, j, s.full[st]);
          for (int nb = 0; nb < nbox; ++nb) tma_load_3d(a + kABytes + nb * 8192, &tmR, nb * 64, kc * 64, j, s.full[st]);
          if (++st == kStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(128, p.C, 1, 1);
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
    const size_t l = (size_t)p.d * p.C;
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int j = tile / p.tiles_per_part, mt = tile % p.tiles_per_part;
      if (!mbar_wait(s.tfull[buf], aph)) { failed = true; break; }
      tc_fence_after();
      const int dcol = mt * 128 + q * 32 + lane;
      const bool valid = dcol < p.d;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 256u;
      float *dst = p.G + (size_t)j * l + (size_t)(valid ? dcol : 0) * p.C;
      float v[32];
      for (int c0 = 0; c0 < p.C; c0 += 32) {
        tmem_ld32(taddr + c0, v);
        if (valid) {
#pragma unroll
          for (int g4 = 0; g4 < 8; ++g4)
            if (c0 + g4 * 4 < p.C)
              *reinterpret_cast<float4 *>(dst + c0 + g4 * 4) = make_float4(v[g4 * 4], v[g4 * 4 + 1], v[g4 * 4 + 2], v[g4 * 4 + 3]);
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
  transpose_to_bf16_kernel<<<tg, tb, 0, stream>>>(W, Wt, d, C);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  TcParams p;
  p.k = k; p.rows = rows; p.d = d; p.C = C;
  p.y = y; p.R = R; p.G = G; p.status = status;

  e = cudaFuncSetAttribute(softmax_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(softmax_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTc);
  if (e != cudaSuccess) return e;

  p.tiles_per_part = (rows + 127) / 128;
  p.num_tiles = k * p.tiles_per_part;
  p.num_k = (d + 63) / 64;
  softmax_fwd_kernel<<<p.num_tiles < sms ? p.num_tiles : sms, kTcThreads, kSmemTc, stream>>>(tmXa, tmW, p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  p.tiles_per_part = (d + 127) / 128;
  p.num_tiles = k * p.tiles_per_part;
  p.num_k = (rows + 63) / 64;
  softmax_bwd_kernel<<<p.num_tiles < sms ? p.num_tiles : sms, kTcThreads, kSmemTc, stream>>>(tmXb, tmR, p);
  return cudaGetLastError();
}

}  // namespace ngc
