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
#include <mutex>
#include <new>
#include <vector>

#include "ngc_device.h"
#include "ngc_pdl.cuh"
#include "ngc_tc.cuh"

namespace ngc {

namespace {

using namespace tc;

constexpr int kStages = 4;     // backward kernel ring
constexpr int kFwdStages = 3;  // forward kernel ring (the rest of shared memory stages the output tile)
constexpr int kABytes = 128 * 64 * 2;  // 16 KB: 128 x 64 bf16
constexpr int kBBytes = 256 * 64 * 2;  // 32 KB: 256 x 64 bf16
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kTcThreads = 192;   // backward kernels: producer, MMA, 4 epilogue warps
constexpr int kFwdThreads = 320;  // forward kernels: producer, MMA, 8 epilogue warps (two per tensor-memory quadrant)
constexpr int kXchBytes = 2 * 2 * 128 * 4;  // row max / row sum exchanged between the two warps of a quadrant
constexpr int kTmemCols = 512;
constexpr int kStageLd = 264;  // bf16 elements per row of the output staging tile (256 + 8: conflict-free 16-byte rows)
constexpr int kStageTileBytes = 128 * kStageLd * 2;
constexpr int kSmemTc = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */ + kXchBytes;
constexpr int kSmemFwd = kFwdStages * kStageBytes + 1024 + 256 + kXchBytes + kStageTileBytes;

// Forward contraction D[128 rows x N] = X_tile[128 x K] * B^T with a fused epilogue.
// Tile = (partition j, block of 128 rows, block nt of 256 output columns).
struct FwdParams {
  int rows;       // rows per partition
  int n_total;    // output columns in all (classes, or hidden units)
  int row_blocks, n_tiles, num_tiles;
  int num_k;      // K chunks of 64
  const int *y;   // class labels (softmax epilogue)
  __nv_bfloat16 *out;  // [k][rows][out_ld]
  int out_ld;
  int ones_col;   // relu epilogue: column that receives 1.0 (followed by 7 zeros); -1 = none
  int *status;
};

// D[M x N] = A^T B per batch, A stored [batch][K][M] and B stored [batch][K][N_total] (both row-major bf16,
// read as M/N-major operands).  Tile = (batch j, 128 rows of M, 256 columns of N_total).  Batches are taken
// last to first: the forward pass that ran just before went first to last, so its last batches are still in L2.
// The single-CTA kernel numbers its tiles M-block-major: a ragged last M block (the bias row of an MLP layer)
// is then what the CTAs of a second round get, not a full tile.
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

// Consecutive mbarriers addressed by index: the address is computed, not looked up (an array of addresses indexed by
// a run-time stage number would live in local memory and cost a load on every wait of the issuing threads).
struct BarArray {
  uint32_t base;
  __device__ __forceinline__ uint32_t operator[](int i) const { return base + 8u * (uint32_t)i; }
};

struct Smem {
  unsigned char *tiles;
  BarArray full, empty, tfull, tempty;
  uint32_t *tmem_slot;
  volatile int *abort_flag;
  float *xch;
  __nv_bfloat16 *stage;  // forward kernels: 128 x kStageLd output staging tile
  int nst;               // ring depth in use
};

__device__ __forceinline__ Smem carve(unsigned char *raw, int nst) {
  Smem s;
  const uint32_t base = smem_u32(raw);
  s.tiles = raw + ((1024u - (base & 1023u)) & 1023u);
  s.nst = nst;
  uint64_t *bars = reinterpret_cast<uint64_t *>(s.tiles + nst * kStageBytes);
  s.full.base = smem_u32(&bars[0]);
  s.empty.base = smem_u32(&bars[kStages]);
  s.tfull.base = smem_u32(&bars[2 * kStages]);
  s.tempty.base = smem_u32(&bars[2 * kStages + 2]);
  s.tmem_slot = reinterpret_cast<uint32_t *>(&bars[2 * kStages + 4]);
  s.abort_flag = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
  s.xch = reinterpret_cast<float *>(s.tiles + nst * kStageBytes + 256);
  s.stage = reinterpret_cast<__nv_bfloat16 *>(s.tiles + nst * kStageBytes + 256 + kXchBytes);
  return s;
}

// Common prologue: barriers, tensor memory.  Returns the tensor-memory base address.
__device__ __forceinline__ uint32_t prologue(const Smem &s, int warp, int epi_threads) {
  if (threadIdx.x == 0) {
    for (int i = 0; i < s.nst; ++i) {
      mbar_init(s.full[i], 1);
      mbar_init(s.empty[i], 1);
    }
    mbar_init(s.tfull[0], 1);
    mbar_init(s.tfull[1], 1);
    mbar_init(s.tempty[0], epi_threads);
    mbar_init(s.tempty[1], epi_threads);
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
// One 32 x 32 tile (bx along C, by along d) by a block of 256 threads.
__device__ __forceinline__ void transpose_tile_to_bf16(const float *__restrict__ W, const float *__restrict__ bias,
                                                       __nv_bfloat16 *__restrict__ Wt, int d, int C, int ld, int bx,
                                                       int by, float (*tile)[33]) {
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int c0 = bx * 32, d0 = by * 32;
  for (int r = ty; r < 32; r += 8) {
    const int dd = d0 + r, c = c0 + tx;
    float v = 0.f;
    if (c < C) {
      if (dd < d) v = W[(size_t)dd * C + c];
      else if (dd == d && bias) v = bias[c];
    }
    tile[r][tx] = v;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int c = c0 + r, dd = d0 + tx;
    if (c < C && dd < ld) Wt[(size_t)c * ld + dd] = __float2bfloat16_rn(tile[tx][r]);
  }
}

__global__ void __launch_bounds__(256)
transpose_to_bf16_kernel(const float *__restrict__ W, const float *__restrict__ bias, __nv_bfloat16 *__restrict__ Wt,
                         int d, int C, int ld) {
  pdl_sync();
  __shared__ float tile[32][33];
  transpose_tile_to_bf16(W, bias, Wt, d, C, ld, blockIdx.x, blockIdx.y, tile);
}

// X (fp32, [rows_total][d]) -> bf16 [rows_total][ld] with a column of ones at index d and zeros after
// it: the ones column turns the bias of the first layer, and the bias gradient, into one more row of
// the weight contraction.  One thread per 8 output columns.
__device__ __forceinline__ void convert_x_block(const float *__restrict__ X, __nv_bfloat16 *__restrict__ Xb,
                                                long long rows_total, int d, int ld, long long block) {
  const int groups = ld / 8;
  const long long idx = block * blockDim.x + threadIdx.x;
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

// Epilogues of the forward contractions.  Two threads share an accumulator row (same tensor-memory lane,
// warps w and w + 4): thread `half` owns the 32-column chunks [c_lo, c_lo + nch), at most 4 of them.  All of
// them are pulled into registers with back-to-back tensor-memory loads and one wait, after which the
// accumulator buffer is handed back to the MMA warp (`release()`), before any arithmetic.
//
// Softmax residual R = softmax(z) - onehot(label), rounded to bf16: row max and row sum are exchanged through
// `xch` ([2][2][128] floats) and a 64-thread named barrier per lane quadrant; one exponential per element.
//
// Failure handling of the forward epilogues: the 256 epilogue threads meet at named barriers, which have no
// time limit, so a thread whose bounded wait gave up must not leave on its own.  It raises the shared abort
// flag and walks on; everybody samples the flag between the tile's two block-wide barriers (`stop`), where
// no thread can be writing it, and all leave together after the second one.
template <typename Release>
__device__ __forceinline__ void softmax_residual_row(uint32_t taddr, int ncol, int c_lo, int nch, int label,
                                                     __nv_bfloat16 *srow, float *xch, int rt, int half, int bar_id,
                                                     Release release, const volatile int *abort_flag, int &stop) {
  constexpr float kLog2e = 1.4426950408889634f;
  uint32_t r[128];
  tmem_ld_chunks<4>(taddr + c_lo * 32, nch, r);
  release();
  const int nmine = min(ncol - c_lo * 32, nch * 32);  // columns of this thread (multiple of 16, may be <= 0)
  float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
  for (int i = 0; i < 128; i += 4) {
    if (i < nmine) {
      m0 = fmaxf(m0, __uint_as_float(r[i]));
      m1 = fmaxf(m1, __uint_as_float(r[i + 1]));
      m2 = fmaxf(m2, __uint_as_float(r[i + 2]));
      m3 = fmaxf(m3, __uint_as_float(r[i + 3]));
    }
  }
  xch[half * 128 + rt] = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
  asm volatile("bar.sync %0, 64;" ::"r"(bar_id) : "memory");
  const float mxs = fmaxf(xch[rt], xch[128 + rt]) * kLog2e;
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int i = 0; i < 128; i += 4) {
    const bool in = i < nmine;
    const float e0 = in ? exp2f(fmaf(__uint_as_float(r[i]), kLog2e, -mxs)) : 0.f;
    const float e1 = in ? exp2f(fmaf(__uint_as_float(r[i + 1]), kLog2e, -mxs)) : 0.f;
    const float e2 = in ? exp2f(fmaf(__uint_as_float(r[i + 2]), kLog2e, -mxs)) : 0.f;
    const float e3 = in ? exp2f(fmaf(__uint_as_float(r[i + 3]), kLog2e, -mxs)) : 0.f;
    s0 += e0; s1 += e1; s2 += e2; s3 += e3;
    r[i] = __float_as_uint(e0); r[i + 1] = __float_as_uint(e1);
    r[i + 2] = __float_as_uint(e2); r[i + 3] = __float_as_uint(e3);
  }
  xch[256 + half * 128 + rt] = (s0 + s1) + (s2 + s3);
  asm volatile("bar.sync %0, 64;" ::"r"(bar_id) : "memory");
  const float inv = 1.f / (xch[256 + rt] + xch[256 + 128 + rt]);
  const int lm = label - c_lo * 32;  // position of the label among this thread's columns
  asm volatile("bar.sync 5, 256;" ::: "memory");  // the previous tile has left the staging buffer
  stop = *abort_flag;
#pragma unroll
  for (int g8 = 0; g8 < 16; ++g8) {  // 8 values = one 16-byte store
    uint32_t w[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const int i = g8 * 8 + h * 2;
      const float r0 = __uint_as_float(r[i]) * inv - (i == lm ? 1.f : 0.f);
      const float r1 = __uint_as_float(r[i + 1]) * inv - (i + 1 == lm ? 1.f : 0.f);
      const __nv_bfloat162 b2 = __floats2bfloat162_rn(r0, r1);
      w[h] = *reinterpret_cast<const uint32_t *>(&b2);
    }
    if (g8 * 8 < nmine) *reinterpret_cast<uint4 *>(srow + c_lo * 32 + g8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// H = relu(z), rounded to bf16.
template <typename Release>
__device__ __forceinline__ void relu_row(uint32_t taddr, int ncol, int c_lo, int nch, __nv_bfloat16 *srow,
                                         Release release, const volatile int *abort_flag, int &stop) {
  uint32_t r[128];
  tmem_ld_chunks<4>(taddr + c_lo * 32, nch, r);
  release();
  const int nmine = min(ncol - c_lo * 32, nch * 32);
  asm volatile("bar.sync 5, 256;" ::: "memory");  // the previous tile has left the staging buffer
  stop = *abort_flag;
#pragma unroll
  for (int g8 = 0; g8 < 16; ++g8) {
    uint32_t w[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const int i = g8 * 8 + h * 2;
      const __nv_bfloat162 b2 =
          __floats2bfloat162_rn(fmaxf(__uint_as_float(r[i]), 0.f), fmaxf(__uint_as_float(r[i + 1]), 0.f));
      w[h] = *reinterpret_cast<const uint32_t *>(&b2);
    }
    if (g8 * 8 < nmine) *reinterpret_cast<uint4 *>(srow + c_lo * 32 + g8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// Copies the staged 128 x ncol bf16 tile to global memory with full-row (coalesced) warp stores: each of the
// 8 epilogue warps takes 16 rows.  `out_row0` points at column 0 of the tile's first row; rows beyond
// `nrows` do not exist.
__device__ __forceinline__ void store_staged_tile(const __nv_bfloat16 *stage, __nv_bfloat16 *out_row0, int out_ld,
                                                  int nrows, int ncol, int epi_warp, int lane) {
  if (lane * 8 < ncol) {
#pragma unroll 4
    for (int rr = epi_warp * 16; rr < epi_warp * 16 + 16; ++rr) {
      if (rr < nrows)
        *reinterpret_cast<uint4 *>(out_row0 + (size_t)rr * out_ld + lane * 8) =
            *reinterpret_cast<const uint4 *>(stage + rr * kStageLd + lane * 8);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Forward contractions.  EPI = 0: softmax residual  R = softmax(Z) - onehot(y)  (needs all classes in one
// tile).  EPI = 1: H = relu(Z) (first MLP layer; bias already folded into the contraction).
// ------------------------------------------------------------------------------------------------
template <int EPI>
__global__ void __launch_bounds__(kFwdThreads, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const FwdParams p) {
  pdl_sync();
  extern __shared__ unsigned char smem_raw[];
  const Smem s = carve(smem_raw, kFwdStages);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_base = prologue(s, warp, kFwdThreads - 64);
  bool failed = false;

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      const uint64_t stream_once = l2_evict_first_policy();  // the data matrix: read once by this kernel
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        const int nt = tile % p.n_tiles, rb = (tile / p.n_tiles) % p.row_blocks, j = tile / (p.n_tiles * p.row_blocks);
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.empty[st], ph ^ 1u)) { failed = true; break; }
          mbar_expect_tx(s.full[st], kStageBytes);
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          tma_load_3d_hint(a, &tmX, kc * 64, rb * 128, j, s.full[st], stream_once);
          tma_load_2d(a + kABytes, &tmW, kc * 64, nt * 256, s.full[st]);
          if (++st == kFwdStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    {  // all 32 lanes walk the loop (uniform operands); one elected lane issues the tensor-core instructions
      int st = 0, buf = 0;
      uint32_t ph = 0, aph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        const int nt = tile % p.n_tiles;
        const uint32_t idesc = instr_desc_bf16(128, min(256, p.n_total - nt * 256), 0, 0);
        if (!mbar_wait_warp(s.tempty[buf], aph ^ 1u)) { failed = true; break; }
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)buf * 256u;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait_warp(s.full[st], ph)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          const uint64_t ad = smem_desc_sw128(a, 16, 1024), bd = smem_desc_sw128(a + kABytes, 16, 1024);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)  // 16 bf16 = 32 bytes along K per instruction
            mma_bf16(acc, ad + (uint64_t)(k4 * 2), bd + (uint64_t)(k4 * 2), idesc, (kc | k4) != 0);
          mma_commit(s.empty[st]);
          if (++st == kFwdStages) { st = 0; ph ^= 1u; }
        }
        if (failed) break;
        mma_commit(s.tfull[buf]);
        buf ^= 1;
        if (buf == 0) aph ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;            // the 32-lane quadrant of tensor memory this warp may read
    const int half = (warp - 2) >> 2;  // warps w and w + 4 share a quadrant and split the columns
    int buf = 0;
    uint32_t aph = 0;
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const int nt = tile % p.n_tiles, rb = (tile / p.n_tiles) % p.row_blocks, j = tile / (p.n_tiles * p.row_blocks);
      if (!mbar_wait(s.tfull[buf], aph)) { failed = true; *s.abort_flag = 1; }
      tc_fence_after();
      int stop = 0;
      const int rt = q * 32 + lane, row = rb * 128 + rt;
      const bool valid = row < p.rows;
      const size_t grow = (size_t)j * p.rows + (valid ? row : 0);
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 256u;
      const int ncol = min(256, p.n_total - nt * 256);
      const int nchunks = (ncol + 31) >> 5, hc = (nchunks + 1) >> 1;
      const int c_lo = half ? hc : 0, nch = half ? nchunks - hc : hc;  // this thread's 32-column chunks
      __nv_bfloat16 *srow = s.stage + rt * kStageLd;
      const uint32_t tempty_bar = s.tempty[buf];
      auto release = [&]() {  // the accumulator values are in registers: the MMA warp may overwrite the buffer
        tc_fence_before();
        mbar_arrive(tempty_bar);
      };
      if (EPI == 0) {
        softmax_residual_row(taddr, ncol, c_lo, nch, valid ? p.y[grow] : -1, srow, s.xch, rt, half, 1 + q, release,
                             s.abort_flag, stop);
      } else {
        relu_row(taddr, ncol, c_lo, nch, srow, release, s.abort_flag, stop);
        if (valid && half == 0 && nt == 0 && p.ones_col >= 0)  // bf16 1.0 followed by zeros
          *reinterpret_cast<uint4 *>(p.out + grow * p.out_ld + p.ones_col) = make_uint4(0x00003f80u, 0u, 0u, 0u);
      }
      asm volatile("bar.sync 5, 256;" ::: "memory");  // the tile is complete in shared memory
      if (stop) break;  // (the same value in all 256 threads)
      store_staged_tile(s.stage, p.out + ((size_t)j * p.rows + rb * 128) * p.out_ld + nt * 256, p.out_ld,
                        p.rows - rb * 128, ncol, warp - 2, lane);
      buf ^= 1;
      if (buf == 0) aph ^= 1u;
    }
  }
  epilogue_teardown(s, warp, tmem_base, failed, p.status);
}

// ------------------------------------------------------------------------------------------------
// MLP head on the CUDA cores (the output layer is 10-wide: no tensor-core shape):
//   z = h W2 + b2,  delta2 = softmax(z) - onehot(y),  delta1 = (delta2 W2^T) * (h > 0).
// h comes as bf16 rows (the forward's output); delta1 is stored as bf16 rows, delta2 as bf16 rows of 64
// (16 used).  A block stages 64 consecutive rows of h in shared memory with coalesced loads; four
// threads share a row (a quarter of the hidden units each), exchange their partial logits through
// shared memory, overwrite h by delta1 in place, and the block copies the tile out coalesced.  W2 sits in
// shared memory, padded to CPAD classes, and is read by broadcast.
// ------------------------------------------------------------------------------------------------
constexpr int kHeadRows = 64;
constexpr int kHeadThreads = 256;

template <int CPAD>
__global__ void __launch_bounds__(kHeadThreads)
mlp_head_kernel(const __nv_bfloat16 *__restrict__ H, int hpad, int hidden, int C, const float *__restrict__ W2,
                const float *__restrict__ b2, const int *__restrict__ y, long long rows_total,
                __nv_bfloat16 *__restrict__ D1, __nv_bfloat16 *__restrict__ D2) {
  pdl_sync();
  extern __shared__ __align__(16) unsigned char head_smem[];
  float *w2s = reinterpret_cast<float *>(head_smem);                 // [hidden][CPAD], then b2[CPAD]
  float *zpart = w2s + (size_t)hidden * CPAD + CPAD;                 // [4][kHeadRows][CPAD]
  uint4 *tile = reinterpret_cast<uint4 *>(zpart + 4 * kHeadRows * CPAD);  // [kHeadRows][hpad / 8]
  const int tid = threadIdx.x;
  for (int e = tid; e < hidden * CPAD; e += kHeadThreads) {
    const int hc = e / CPAD, c = e % CPAD;
    w2s[e] = c < C ? W2[(size_t)hc * C + c] : 0.f;
  }
  if (tid < CPAD) w2s[hidden * CPAD + tid] = tid < C ? b2[tid] : 0.f;
  const long long row0 = (long long)blockIdx.x * kHeadRows;
  const int nrows = (int)min((long long)kHeadRows, rows_total - row0);
  const int gpr = hpad / 8, hg = hidden / 8;  // 16-byte groups per stored row / per row of hidden units
  {
    const uint4 *src = reinterpret_cast<const uint4 *>(H + row0 * hpad);
    for (int e = tid; e < nrows * gpr; e += kHeadThreads) tile[e] = __ldg(src + e);
  }
  __syncthreads();
  const int part = tid >> 6, r = tid & 63;
  const int gper = (hg + 3) / 4, g_begin = part * gper, g_end = min(hg, g_begin + gper);
  const bool valid = r < nrows;
  float z[CPAD];
#pragma unroll
  for (int c = 0; c < CPAD; ++c) z[c] = 0.f;
  if (valid) {
    for (int g8 = g_begin; g8 < g_end; ++g8) {
      const uint4 u = tile[r * gpr + g8];
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float h = __uint_as_float((i & 1) ? (w[i >> 1] & 0xffff0000u) : (w[i >> 1] << 16));
        const float4 *w2 = reinterpret_cast<const float4 *>(w2s + (size_t)(g8 * 8 + i) * CPAD);
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
  for (int c = 0; c < CPAD; ++c) zpart[(part * kHeadRows + r) * CPAD + c] = z[c];
  __syncthreads();
  float dl[CPAD];
  {
    float mx = -INFINITY;
#pragma unroll
    for (int c = 0; c < CPAD; ++c) {
      z[c] = zpart[r * CPAD + c] + zpart[(kHeadRows + r) * CPAD + c] + zpart[(2 * kHeadRows + r) * CPAD + c] +
             zpart[(3 * kHeadRows + r) * CPAD + c] + w2s[hidden * CPAD + c];
      if (c < C) mx = fmaxf(mx, z[c]);
    }
    float sum = 0.f;
#pragma unroll
    for (int c = 0; c < CPAD; ++c) {
      dl[c] = c < C ? __expf(z[c] - mx) : 0.f;
      sum += dl[c];
    }
    const float inv = 1.f / sum;
    const int label = valid ? y[row0 + r] : -1;
#pragma unroll
    for (int c = 0; c < CPAD; ++c) dl[c] = c < C ? dl[c] * inv - (c == label ? 1.f : 0.f) : 0.f;
  }
  if (valid && part == 0) {
    uint32_t w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float lo = 2 * i < CPAD ? dl[2 * i < CPAD ? 2 * i : 0] : 0.f;
      const float hi = 2 * i + 1 < CPAD ? dl[2 * i + 1 < CPAD ? 2 * i + 1 : 0] : 0.f;
      const __nv_bfloat162 b2v = __floats2bfloat162_rn(lo, hi);
      w[i] = *reinterpret_cast<const uint32_t *>(&b2v);
    }
    uint4 *d2 = reinterpret_cast<uint4 *>(D2 + (row0 + r) * 64);
    d2[0] = make_uint4(w[0], w[1], w[2], w[3]);
    d2[1] = make_uint4(w[4], w[5], w[6], w[7]);
  }
  if (valid) {
    for (int g8 = g_begin; g8 < g_end; ++g8) {
      const uint4 u = tile[r * gpr + g8];
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
      uint32_t o[4];
#pragma unroll
      for (int hh = 0; hh < 4; ++hh) {
        float dv[2];
#pragma unroll
        for (int uu = 0; uu < 2; ++uu) {
          const uint32_t bits = uu ? (w[hh] & 0xffff0000u) : (w[hh] << 16);
          const float4 *w2 = reinterpret_cast<const float4 *>(w2s + (size_t)(g8 * 8 + hh * 2 + uu) * CPAD);
          float acc = 0.f;
#pragma unroll
          for (int c4 = 0; c4 < CPAD / 4; ++c4) {
            const float4 ww = w2[c4];
            acc = fmaf(dl[c4 * 4], ww.x, acc);
            acc = fmaf(dl[c4 * 4 + 1], ww.y, acc);
            acc = fmaf(dl[c4 * 4 + 2], ww.z, acc);
            acc = fmaf(dl[c4 * 4 + 3], ww.w, acc);
          }
          dv[uu] = __uint_as_float(bits) > 0.f ? acc : 0.f;
        }
        const __nv_bfloat162 db = __floats2bfloat162_rn(dv[0], dv[1]);
        o[hh] = *reinterpret_cast<const uint32_t *>(&db);
      }
      tile[r * gpr + g8] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  __syncthreads();
  {
    uint4 *dst = reinterpret_cast<uint4 *>(D1 + row0 * hidden);
    for (int e = tid; e < nrows * hg; e += kHeadThreads) dst[e] = tile[(e / hg) * gpr + (e % hg)];
  }
}

// ------------------------------------------------------------------------------------------------
// MLP head on the tensor cores (hidden a multiple of 64, at most 512; at most 16 classes).  Per tile of
// 128 samples of one partition, everything stays in shared / tensor memory:
//   1. TMA brings the 128 x hidden tile of h (bf16, K-major, 128-byte swizzle), in groups of four 64-column chunks;
//   2. z[128 x 16] = h W2 (W2^T resident in shared memory as the B operand, N = 16);
//   3. one thread per sample: z + b2 -> softmax -> delta2, which, as a bf16 row of a swizzled 128 x 64 tile,
//      becomes an operand of the next contractions;
//   4. hidden a multiple of 128: dW2 += h^T delta2 (samples as K: both tiles read M/N-major), accumulated in
//      tensor memory over the CTA's tiles of a partition; db2 by warp shuffles.  Otherwise delta2 goes to
//      global memory and a backward contraction forms dW2;
//   5. (delta2 W2^T)[128 x hidden] with K = 16: one MMA per 256 hidden units;
//   6. the threads mask by h > 0 (read from the tile in its swizzled layout) and overwrite h by delta1 in
//      place; the producer stores each finished group to delta1[rows][hidden] and reloads it with the next
//      tile's h while the other group is still being worked on.
// ------------------------------------------------------------------------------------------------
constexpr int kHeadEpiThreads = 512;  // 16 epilogue warps: four per tensor-memory quadrant
constexpr int kHeadTcThreads = 96 + kHeadEpiThreads;  // + two producer warps and the MMA warp

struct HeadTcParams {
  int hidden, C, rows, tiles_per_part, num_tiles;  // a tile = 128 rows of one partition
  const float *b2;
  const int *y;
  __nv_bfloat16 *D2;  // [k * rows][64]: delta2 rows, written only when the output-layer gradient is formed elsewhere
  int fuse;           // 1: [dW2; db2] = [h 1]^T delta2 is formed here (hidden a multiple of 128)
  float *slots;       // [k][max_slots][hidden * C + C]: partial sums of the CTAs that share a partition
  int max_slots;
  int *status;
};

// Tiles [begin, end) of CTA c when `tiles` tiles are cut into `grid` contiguous ranges.
__host__ __device__ inline int head_tile_begin(int c, int tiles, int grid) { return (int)((long long)c * tiles / grid); }

__device__ __forceinline__ void prep_w2_block(const float *__restrict__ W2, int hidden, int C,
                                              __nv_bfloat16 *__restrict__ W2t, __nv_bfloat16 *__restrict__ W2k, int block) {
  const int i = block * blockDim.x + threadIdx.x;
  if (i < 16 * hidden) {  // W2t[c][hc]
    const int c = i / hidden, hc = i % hidden;
    W2t[i] = __float2bfloat16_rn(c < C ? W2[(size_t)hc * C + c] : 0.f);
  }
  if (i < hidden * 64) {  // W2k[hc][c]
    const int hc = i / 64, c = i % 64;
    W2k[i] = __float2bfloat16_rn(c < C ? W2[(size_t)hc * C + c] : 0.f);
  }
}

// Everything the MLP gradient needs before its first contraction, in one launch of 256-thread blocks: the
// data matrix as bf16 with a column of ones (the bulk of the blocks, bound by HBM), W1 / b1 transposed to the
// K-major operand of the forward contraction, and (w2_blocks > 0) the two layouts of W2 the head reads.  The
// small jobs sit at the front of the grid and finish under the conversion.
struct MlpPrepParams {
  const float *X; __nv_bfloat16 *Xb; long long rows_total; int d, dpad;
  const float *W1, *b1; __nv_bfloat16 *W1t; int hidden;
  const float *W2; int C; __nv_bfloat16 *W2t, *W2k;
  int tr_bx, tr_blocks, w2_blocks;
};

__global__ void __launch_bounds__(256) mlp_prep_kernel(const MlpPrepParams p) {
  pdl_sync();
  __shared__ float tile[32][33];
  int b = blockIdx.x;
  if (b < p.tr_blocks) {
    transpose_tile_to_bf16(p.W1, p.b1, p.W1t, p.d, p.hidden, p.dpad, b % p.tr_bx, b / p.tr_bx, tile);
    return;
  }
  b -= p.tr_blocks;
  if (b < p.w2_blocks) {
    prep_w2_block(p.W2, p.hidden, p.C, p.W2t, p.W2k, b);
    return;
  }
  b -= p.w2_blocks;
  convert_x_block(p.X, p.Xb, p.rows_total, p.d, p.dpad, b);
}

__global__ void __launch_bounds__(kHeadTcThreads, 1)
mlp_head_tc_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW2t,
                   const __grid_constant__ CUtensorMap tmW2k, const __grid_constant__ CUtensorMap tmD1,
                   const HeadTcParams p) {
  pdl_sync();
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char *sm = smem_raw + ((1024u - (base & 1023u)) & 1023u);
  const int nchunk = p.hidden / 64, nhalf = (p.hidden + 255) / 256, ngroups = nchunk;
  unsigned char *htile = sm;                                  // nchunk x [128 x 64] bf16
  unsigned char *d2tile = htile + (size_t)nchunk * 16384;     // [128 x 64] bf16 (16 columns used)
  unsigned char *w2k = d2tile + 16384;                        // nhalf x [256 x 64] bf16
  unsigned char *w2t = w2k + (size_t)nhalf * 32768;           // nchunk x [16 x 64] bf16
  uint64_t *bars = reinterpret_cast<uint64_t *>(w2t + (size_t)nchunk * 2048);
  // The tile lives in shared memory as 64-column chunks.  Chunk g is loaded (h), consumed, overwritten in place
  // (delta1), stored and reloaded with the next tile's h on its own barriers, so the memory traffic of the
  // finished chunks hides behind the arithmetic on the others, and what is left when the last chunk is done is
  // one chunk's store and reload (with pairs of chunks it was two chunks' worth: a quarter of the tile's time).
  const BarArray h_full{smem_u32(&bars[0])}, m_done{smem_u32(&bars[8])}, w_done{smem_u32(&bars[16])};
  const uint32_t z_full = smem_u32(&bars[20]), d2_full = smem_u32(&bars[21]), d_full = smem_u32(&bars[22]),
                 d_empty = smem_u32(&bars[23]), w_full = smem_u32(&bars[24]);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(&bars[25]);
  float *b2s = reinterpret_cast<float *>(&bars[26]);          // 16 floats
  float *dbx = reinterpret_cast<float *>(&bars[34]);          // [4 quadrants][16]: bias-gradient partial sums
  const uint32_t epi_bar = smem_u32(&bars[66]);               // meeting point of the epilogue threads (bounded, unlike bar.sync)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      mbar_init(h_full[g], 1);
      mbar_init(m_done[g], kHeadEpiThreads);
      if (g < 4) mbar_init(w_done[g], 1);
    }
    mbar_init(z_full, 1);
    mbar_init(d2_full, 128);
    mbar_init(d_full, 1);
    mbar_init(d_empty, kHeadEpiThreads);
    mbar_init(w_full, 1);
    mbar_init(epi_bar, kHeadEpiThreads);
    mbar_fence_init();
  }
  if (threadIdx.x < 16) b2s[threadIdx.x] = (int)threadIdx.x < p.C ? p.b2[threadIdx.x] : 0.f;
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t z_acc = tmem_base, w2_acc = tmem_base + 32u, d_acc = tmem_base + 256u;
  bool failed = false;
  const int grid = (int)gridDim.x, tpp = p.tiles_per_part;
  const int t_begin = head_tile_begin((int)blockIdx.x, p.num_tiles, grid),
            t_end = head_tile_begin((int)blockIdx.x + 1, p.num_tiles, grid);

  if (warp == 0 || warp == 2) {
    // Two producers: warp 0 owns the even chunks, warp 2 the odd ones, so that one of them can wait for a store to
    // release its chunk while the other already handles the next chunk.
    if (lane == 0) {
      const int g0 = warp >> 1;
      if (warp == 0) {
        mbar_expect_tx(w_full, (uint32_t)(nchunk * 2048 + nhalf * 32768));
        for (int kc = 0; kc < nchunk; ++kc) tma_load_2d(smem_u32(w2t + kc * 2048), &tmW2t, kc * 64, 0, w_full);
        for (int hh = 0; hh < nhalf; ++hh) tma_load_2d(smem_u32(w2k + hh * 32768), &tmW2k, 0, hh * 256, w_full);
      }
      const uint64_t stream_once = l2_evict_first_policy();  // h is read here for the last time
      auto load_group = [&](int tile, int g) {
        const int j = tile / tpp, rb = tile % tpp;
        mbar_expect_tx(h_full[g], 16384u);
        tma_load_3d_hint(smem_u32(htile + g * 16384), &tmH, g * 64, rb * 128, j, h_full[g], stream_once);
      };
      for (int g = g0; g < ngroups; g += 2) load_group(t_begin, g);
      uint32_t ph = 0;
      for (int tile = t_begin; tile < t_end && !failed; ++tile) {
        const int j = tile / tpp, rb = tile % tpp;
        for (int g = g0; g < ngroups; g += 2) {
          // delta1 has replaced h in chunk g: store it, and once the store has read shared memory bring the
          // next tile's h into the same chunk
          if (!mbar_wait(m_done[g], ph)) { failed = true; break; }
          tma_store_3d(&tmD1, g * 64, rb * 128, j, smem_u32(htile + g * 16384));
          tma_store_commit_and_wait_read();
          if (tile + 1 < t_end) load_group(tile + 1, g);
        }
        ph ^= 1u;
      }
    }
  } else if (warp == 1) {
    {  // all 32 lanes walk the loop (uniform operands); one elected lane issues the tensor-core instructions
      const uint32_t idesc_z = instr_desc_bf16(128, 16, 0, 0), idesc_w = instr_desc_bf16(128, 16, 1, 1);
      const int nmb = p.hidden / 128;
      uint32_t ph = 0, dph = 0;
      if (!mbar_wait_warp(w_full, 0)) failed = true;
      for (int tile = t_begin; tile < t_end && !failed; ++tile) {
        for (int g = 0; g < ngroups && !failed; ++g) {
          if (!mbar_wait_warp(h_full[g], ph)) { failed = true; break; }
          tc_fence_after();
          {
            const int kc = g;
            const uint64_t ad = smem_desc_sw128(smem_u32(htile + kc * 16384), 16, 1024);
            const uint64_t bd = smem_desc_sw128(smem_u32(w2t + kc * 2048), 16, 1024);
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4)
              mma_bf16(z_acc, ad + (uint64_t)(k4 * 2), bd + (uint64_t)(k4 * 2), idesc_z, (kc | k4) != 0);
          }
        }
        if (failed) break;
        mma_commit(z_full);
        if (!mbar_wait_warp(d2_full, ph)) { failed = true; break; }
        tc_fence_after();
        const bool first = tile == t_begin || tile % tpp == 0;  // first tile of its partition in this CTA
        const uint64_t ad1 = smem_desc_sw128(smem_u32(d2tile), 16, 1024);      // delta2, K-major (K = classes)
        const uint64_t bdw = smem_desc_sw128(smem_u32(d2tile), 16384, 1024);   // delta2, N-major (K = samples)
        for (int hh = 0; hh < nhalf; ++hh) {
          if (!mbar_wait_warp(d_empty, dph ^ 1u)) { failed = true; break; }
          tc_fence_after();
          const int nh = min(256, p.hidden - hh * 256);
          const uint64_t bd = smem_desc_sw128(smem_u32(w2k + hh * 32768), 16, 1024);
          mma_bf16(d_acc, ad1, bd, instr_desc_bf16(128, nh, 0, 0), 0);  // K = 16: the 16 class columns
          mma_commit(d_full);
          dph ^= 1u;
          if (p.fuse) {
            // dW2 block (128 hidden units x 16 classes) += h_block^T delta2 for the two blocks inside this half:
            // both operands are read M/N-major from the tiles the other contractions use K-major.  They run
            // while the epilogue fetches the delta1 accumulator; block mb = chunk group mb may be overwritten
            // once w_done[mb] has fired.
            for (int mb = hh * 2; mb < min(nmb, hh * 2 + 2); ++mb) {
              const uint64_t adw = smem_desc_sw128(smem_u32(htile + mb * 32768), 16384, 1024);
#pragma unroll
              for (int k8 = 0; k8 < 8; ++k8)  // 16 samples = 2048 bytes per instruction
                mma_bf16(w2_acc + (uint32_t)mb * 16u, adw + (uint64_t)(k8 * 128), bdw + (uint64_t)(k8 * 128), idesc_w,
                         !(first && k8 == 0));
              mma_commit(w_done[mb]);
            }
          }
        }
        ph ^= 1u;
      }
    }
  } else {
    const int q = warp & 3, r = q * 32 + lane;  // row of the tile = tensor-memory lane
    const int part = (warp - 3) >> 2;           // the four warps of a quadrant split every chunk: 16 columns each
    const int tid_epi = (int)threadIdx.x - 96;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t row_off = (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u;  // row r inside a swizzled tile
    const uint32_t rx = (uint32_t)(r & 7);
    const int wstride = p.hidden * p.C + p.C;
    uint32_t ph = 0, dph = 0, eph = 0;
    // all epilogue threads meet: arrive, then a bounded wait for the others (a thread that gave up elsewhere
    // never arrives, and the rest then give up here instead of waiting for ever)
    auto epi_sync = [&]() -> bool {
      mbar_arrive(epi_bar);
      const bool ok = mbar_wait(epi_bar, eph);
      eph ^= 1u;
      return ok;
    };
    float db2_acc = 0.f;  // lane c of a part-0 warp: sum of delta2[., c] over the warp's rows
    for (int tile = t_begin; tile < t_end; ++tile) {
      const int j = tile / tpp, rb = tile % tpp;
      const int prow = rb * 128 + r;
      const bool valid = prow < p.rows;
      const long long row = (long long)j * p.rows + prow;
      if (part == 0) {
        const int label = valid ? __ldg(p.y + row) : -1;  // on its way while the logits are being formed
        if (!mbar_wait(z_full, ph)) { failed = true; break; }
        tc_fence_after();
        float v[16];
        tmem_ld16(z_acc + lane_off, v);
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          v[c] += b2s[c];
          if (c < p.C) mx = fmaxf(mx, v[c]);
        }
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          v[c] = c < p.C ? __expf(v[c] - mx) : 0.f;
          sum += v[c];
        }
        const float inv = valid ? 1.f / sum : 0.f;  // rows beyond the partition contribute nothing
        uint32_t w[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float lo = (2 * u < p.C) ? v[2 * u] * inv - (2 * u == label ? 1.f : 0.f) : 0.f;
          const float hi = (2 * u + 1 < p.C) ? v[2 * u + 1] * inv - (2 * u + 1 == label ? 1.f : 0.f) : 0.f;
          const __nv_bfloat162 b2v = __floats2bfloat162_rn(lo, hi);
          w[u] = *reinterpret_cast<const uint32_t *>(&b2v);
        }
        *reinterpret_cast<uint4 *>(d2tile + row_off + ((0u ^ rx) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4 *>(d2tile + row_off + ((1u ^ rx) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
        fence_async_smem();
        mbar_arrive(d2_full);
        if (valid && !p.fuse) {
          uint4 *d2 = reinterpret_cast<uint4 *>(p.D2 + row * 64);
          d2[0] = make_uint4(w[0], w[1], w[2], w[3]);
          d2[1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
        if (p.fuse) {  // db2: column sums of the rounded delta2 over this warp's 32 rows, class c kept by lane c
          float mine = 0.f;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            float t = __uint_as_float((c & 1) ? (w[c >> 1] & 0xffff0000u) : (w[c >> 1] << 16));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == c) mine = t;
          }
          db2_acc += mine;
        }
      }
      uint32_t rr[64];  // this thread's 16 columns of each of the (up to) four chunks of a 256-column half
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        if (g >= ngroups || failed) break;
        // the threads read h themselves below: observe the completion of its TMA copies directly
        if (!mbar_wait(h_full[g], ph)) { failed = true; break; }
        if ((g & 3) == 0) {  // first chunk of a half: fetch the half's accumulator and hand it back at once
          if (!mbar_wait(d_full, dph)) { failed = true; break; }
          tc_fence_after();
          const int hh = g >> 2, nlc = min(4, nchunk - hh * 4);
#pragma unroll
          for (int lc = 0; lc < 4; ++lc)
            if (lc < nlc) tmem_ld16_nowait(d_acc + lane_off + (uint32_t)(lc * 64 + part * 16), &rr[lc * 16]);
          tmem_ld_wait(rr);
          tc_fence_before();
          mbar_arrive(d_empty);
          dph ^= 1u;
        }
        // the tensor cores are done with the 128 hidden units (two chunks) this chunk belongs to
        if (p.fuse && (g & 1) == 0 && !mbar_wait(w_done[g >> 1], ph)) { failed = true; break; }
        const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
        {
          const int kc = g;  // chunk of 64 hidden units
          {
            unsigned char *crow = htile + (size_t)kc * 16384 + row_off;
            uint4 hv[2];
#pragma unroll
            for (int i = 0; i < 2; ++i)
              hv[i] = *reinterpret_cast<const uint4 *>(crow + ((((uint32_t)(part * 2 + i)) ^ rx) << 4));
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              const uint32_t hw4[4] = {hv[i].x, hv[i].y, hv[i].z, hv[i].w};
              uint32_t o[4];
#pragma unroll
              for (int t2 = 0; t2 < 4; ++t2) {
                // g & 3 = chunk inside the half; delta1 = (h > 0) ? value : 0 as a bf16 pair
                const int e = ((g & 3) * 16) + i * 8 + t2 * 2;
                const __nv_bfloat162 dv = __floats2bfloat162_rn(__uint_as_float(rr[e]), __uint_as_float(rr[e + 1]));
                const __nv_bfloat162 hb = *reinterpret_cast<const __nv_bfloat162 *>(&hw4[t2]);
                const __nv_bfloat162 dm = __hmul2(dv, __hgt2(hb, zero2));
                o[t2] = *reinterpret_cast<const uint32_t *>(&dm);
              }
              *reinterpret_cast<uint4 *>(crow + ((((uint32_t)(part * 2 + i)) ^ rx) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
        }
        fence_async_smem();
        mbar_arrive(m_done[g]);  // this thread's share of delta1 sits where h was
      }
      if (failed) break;
      ph ^= 1u;

      if (p.fuse && (tile + 1 == t_end || (tile + 1) % tpp == 0)) {
        // Last tile of partition j in this CTA: deliver this CTA's share of [dW2; db2] to its slot.  Every
        // tensor-core instruction of the tile has completed (the wait on w_done of the last group above).
        // `head_reduce_kernel` adds up the slots of a partition in CTA order.
        int cfirst = (int)blockIdx.x;
        while (cfirst > 0 && head_tile_begin(cfirst, p.num_tiles, grid) > j * tpp) --cfirst;
        float *dst = p.slots + ((size_t)j * p.max_slots + ((int)blockIdx.x - cfirst)) * wstride;
        if (part == 0) {
          for (int mb = 0; mb < p.hidden / 128; ++mb) {
            float v[16];
            tmem_ld16(w2_acc + lane_off + (uint32_t)mb * 16u, v);
            float *o = dst + (size_t)(mb * 128 + r) * p.C;
#pragma unroll
            for (int c = 0; c < 16; ++c)
              if (c < p.C) o[c] = v[c];
          }
          tc_fence_before();
          if (lane < 16) dbx[q * 16 + lane] = db2_acc;
          db2_acc = 0.f;
        }
        if (!epi_sync()) { failed = true; break; }
        if (tid_epi < p.C)
          dst[(size_t)p.hidden * p.C + tid_epi] = (dbx[tid_epi] + dbx[16 + tid_epi]) + (dbx[32 + tid_epi] + dbx[48 + tid_epi]);
        if (!epi_sync()) { failed = true; break; }  // dbx is free again
      }
    }
  }
  if (failed) atomicExch(p.status, 1);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// [dW2; db2] of partition j = sum of the slots the head kernel's CTAs filled, in CTA order (reruns are
// bit-identical).  blockIdx.y = partition.
struct HeadSlots {
  const float *slots;  // [k][max_slots][wstride]; nullptr = nothing to add up
  int max_slots, wstride, tpp, num_tiles, grid, k;
  float *G;            // [dW2; db2] of partition j goes to G + j * g_batch
  size_t g_batch;
};

// Element e of [dW2; db2] of partition j.
__device__ __forceinline__ void head_reduce_one(const HeadSlots &h, int j, int e) {
  // CTAs of the head kernel whose tile range meets partition j
  const int cfirst = (int)(((long long)(j * h.tpp + 1) * h.grid - 1) / h.num_tiles);
  const int clast = (int)(((long long)((j + 1) * h.tpp) * h.grid - 1) / h.num_tiles);
  const float *s0 = h.slots + (size_t)j * h.max_slots * h.wstride + e;
  const int nsl = clast - cfirst + 1;
  float acc = 0.f;
  for (int sb = 0; sb < nsl; sb += 8) {  // eight loads in flight, added in slot order
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = sb + i < nsl ? __ldg(s0 + (size_t)(sb + i) * h.wstride) : 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc += v[i];
  }
  h.G[(size_t)j * h.g_batch + e] = acc;
}

__global__ void head_reduce_kernel(const HeadSlots h) {
  pdl_sync();
  const int j = blockIdx.y, e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e < h.wstride) head_reduce_one(h, j, e);
}

// ------------------------------------------------------------------------------------------------
// Backward contractions: D = A^T B with K = the partition's rows (see TnParams).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTcThreads, 1)
tn_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TnParams p) {
  pdl_sync();
  extern __shared__ unsigned char smem_raw[];
  const Smem s = carve(smem_raw, kStages);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_base = prologue(s, warp, kTcThreads - 64);
  bool failed = false;

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      const uint32_t tx = (uint32_t)(2 + p.nbox) * 8192u;
      const uint64_t stream_once = l2_evict_first_policy();  // the M-side operand (data matrix / activations)
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        const int nt = tile % p.n_tiles, j = p.batch - 1 - (tile / p.n_tiles) % p.batch, mt = tile / (p.n_tiles * p.batch);
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.empty[st], ph ^ 1u)) { failed = true; break; }
          mbar_expect_tx(s.full[st], tx);
          const uint32_t a = smem_u32(s.tiles + st * kStageBytes);
          tma_load_3d_hint(a, &tmA, mt * 128, kc * 64, j, s.full[st], stream_once);
          tma_load_3d_hint(a + 8192, &tmA, mt * 128 + 64, kc * 64, j, s.full[st], stream_once);
          for (int nb = 0; nb < p.nbox; ++nb)
            tma_load_3d(a + kABytes + nb * 8192, &tmB, nt * 256 + nb * 64, kc * 64, j, s.full[st]);
          if (++st == kStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    {  // all 32 lanes walk the loop (uniform operands); one elected lane issues the tensor-core instructions
      const uint32_t idesc = instr_desc_bf16(128, p.N, 1, 1);
      int st = 0, buf = 0;
      uint32_t ph = 0, aph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles && !failed; tile += gridDim.x) {
        if (!mbar_wait_warp(s.tempty[buf], aph ^ 1u)) { failed = true; break; }
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)buf * 256u;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait_warp(s.full[st], ph)) { failed = true; break; }
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
      const int nt = tile % p.n_tiles, j = p.batch - 1 - (tile / p.n_tiles) % p.batch, mt = tile / (p.n_tiles * p.batch);
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
// CTA-pair versions.  Two CTAs of a cluster (two SMs) drive one 256-row MMA (cta_group::2): each loads
// its own 128 rows of A and only HALF of the 256-wide B tile, so the operand bytes an SM pulls from L2
// per tensor-pipe cycle drop from 48 KB / 512 cycles to 32 KB / 512 cycles.  The leader CTA (cluster
// rank 0) issues the MMAs for both; each CTA keeps its 128 accumulator rows in its own tensor memory and
// runs its own epilogue.  Barriers: `full` lives in the leader and collects the TMA bytes of both CTAs;
// `empty` and `tfull` exist in both and are signalled by a multicast commit; `tempty` lives in the leader
// and counts the epilogue threads of both CTAs.
// ------------------------------------------------------------------------------------------------
constexpr int kPairStages = 4;
constexpr int kPairStageBytes = 2 * 16384;  // 128 x 64 of A + 128 x 64 of B
constexpr int kSmemPair = kPairStages * kPairStageBytes + 1024 + 256 + kXchBytes + kStageTileBytes;

struct PairSmem {
  unsigned char *tiles;
  BarArray full, empty, tfull, tempty;
  uint32_t *tmem_slot;
  volatile int *abort_flag;
  float *xch;
  __nv_bfloat16 *stage;
};

__device__ __forceinline__ PairSmem carve_pair(unsigned char *raw) {
  PairSmem s;
  const uint32_t base = smem_u32(raw);
  s.tiles = raw + ((1024u - (base & 1023u)) & 1023u);
  uint64_t *bars = reinterpret_cast<uint64_t *>(s.tiles + kPairStages * kPairStageBytes);
  s.full.base = smem_u32(&bars[0]);
  s.empty.base = smem_u32(&bars[kPairStages]);
  s.tfull.base = smem_u32(&bars[2 * kPairStages]);
  s.tempty.base = smem_u32(&bars[2 * kPairStages + 2]);
  s.tmem_slot = reinterpret_cast<uint32_t *>(&bars[2 * kPairStages + 4]);
  s.abort_flag = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
  s.xch = reinterpret_cast<float *>(s.tiles + kPairStages * kPairStageBytes + 256);
  s.stage = reinterpret_cast<__nv_bfloat16 *>(s.tiles + kPairStages * kPairStageBytes + 256 + kXchBytes);
  return s;
}

__device__ __forceinline__ uint32_t pair_prologue(const PairSmem &s, int warp, int epi_threads) {
  if (threadIdx.x == 0) {
    for (int i = 0; i < kPairStages; ++i) {
      mbar_init(s.full[i], 1);
      mbar_init(s.empty[i], 1);
    }
    mbar_init(s.tfull[0], 1);
    mbar_init(s.tfull[1], 1);
    mbar_init(s.tempty[0], 2 * epi_threads);
    mbar_init(s.tempty[1], 2 * epi_threads);
    *s.abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(s.tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything is signalled on them
  tc_fence_after();
  return *s.tmem_slot;
}

__device__ __forceinline__ void pair_teardown(int warp, uint32_t tmem_base, bool failed, int *status) {
  if (failed) atomicExch(status, 1);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves while the other may still touch its shared or tensor memory
  if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

template <int EPI>
__global__ void __launch_bounds__(kFwdThreads, 1)
fwd_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const FwdParams p) {
  pdl_sync();
  extern __shared__ unsigned char smem_raw[];
  const PairSmem s = carve_pair(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const uint32_t tmem_base = pair_prologue(s, warp, kFwdThreads - 64);
  bool failed = false;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  // p.row_blocks counts 256-row blocks here; this CTA owns rows [rb*256 + rank*128, +128)

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      const uint64_t stream_once = l2_evict_first_policy();  // the data matrix: read once by this kernel
      for (int tile = pair_id; tile < p.num_tiles && !failed; tile += n_pairs) {
        const int nt = tile % p.n_tiles, rb = (tile / p.n_tiles) % p.row_blocks, j = tile / (p.n_tiles * p.row_blocks);
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(s.empty[st], ph ^ 1u)) { failed = true; break; }
          if (rank == 0) mbar_expect_tx(s.full[st], 2 * kPairStageBytes);
          const uint32_t a = smem_u32(s.tiles + st * kPairStageBytes);
          const uint32_t bar = map_to_rank(s.full[st], 0);
          tma_load_3d_pair_hint(a, &tmX, kc * 64, rb * 256 + (int)rank * 128, j, bar, stream_once);
          tma_load_2d_pair(a + 16384, &tmW, kc * 64, nt * 256 + (int)rank * 128, bar);
          if (++st == kPairStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0) {  // all 32 lanes walk the loop (uniform operands); one elected lane issues
      const uint32_t idesc = instr_desc_bf16(256, 256, 0, 0);
      int st = 0, buf = 0;
      uint32_t ph = 0, aph = 0;
      for (int tile = pair_id; tile < p.num_tiles && !failed; tile += n_pairs) {
        if (!mbar_wait_warp(s.tempty[buf], aph ^ 1u)) { failed = true; break; }
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)buf * 256u;
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait_warp(s.full[st], ph)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(s.tiles + st * kPairStageBytes);
          const uint64_t ad = smem_desc_sw128(a, 16, 1024), bd = smem_desc_sw128(a + 16384, 16, 1024);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            mma_bf16_pair(acc, ad + (uint64_t)(k4 * 2), bd + (uint64_t)(k4 * 2), idesc, (kc | k4) != 0);
          mma_commit_pair(s.empty[st], 3);
          if (++st == kPairStages) { st = 0; ph ^= 1u; }
        }
        if (failed) break;
        mma_commit_pair(s.tfull[buf], 3);
        buf ^= 1;
        if (buf == 0) aph ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    int buf = 0;
    uint32_t aph = 0;
    for (int tile = pair_id; tile < p.num_tiles; tile += n_pairs) {
      const int nt = tile % p.n_tiles, rb = (tile / p.n_tiles) % p.row_blocks, j = tile / (p.n_tiles * p.row_blocks);
      if (!mbar_wait(s.tfull[buf], aph)) { failed = true; *s.abort_flag = 1; }
      tc_fence_after();
      int stop = 0;
      const int rt = q * 32 + lane, row = rb * 256 + (int)rank * 128 + rt;
      const bool valid = row < p.rows;
      const size_t grow = (size_t)j * p.rows + (valid ? row : 0);
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 256u;
      const int c_lo = half ? 4 : 0;  // this thread's four 32-column chunks of the 256
      __nv_bfloat16 *srow = s.stage + rt * kStageLd;
      const uint32_t tempty_bar = map_to_rank(s.tempty[buf], 0);
      auto release = [&]() {
        tc_fence_before();
        mbar_arrive_cluster(tempty_bar);
      };
      if (EPI == 0) {
        softmax_residual_row(taddr, 256, c_lo, 4, valid ? p.y[grow] : -1, srow, s.xch, rt, half, 1 + q, release,
                             s.abort_flag, stop);
      } else {
        relu_row(taddr, 256, c_lo, 4, srow, release, s.abort_flag, stop);
        if (valid && half == 0 && nt == 0 && p.ones_col >= 0)
          *reinterpret_cast<uint4 *>(p.out + grow * p.out_ld + p.ones_col) = make_uint4(0x00003f80u, 0u, 0u, 0u);
      }
      asm volatile("bar.sync 5, 256;" ::: "memory");
      if (stop) break;  // (the same value in all 256 threads)
      store_staged_tile(s.stage, p.out + ((size_t)j * p.rows + rb * 256 + (int)rank * 128) * p.out_ld + nt * 256,
                        p.out_ld, p.rows - rb * 256 - (int)rank * 128, 256, warp - 2, lane);
      buf ^= 1;
      if (buf == 0) aph ^= 1u;
    }
  }
  pair_teardown(warp, tmem_base, failed, p.status);
}

// ------------------------------------------------------------------------------------------------
// Wide backward contraction on a CTA pair, roles swapped: D^T = A^T B with A [batch][K][M] on the M side in
// blocks of 256 (128 per CTA) and B [batch][K][n_total] on the N side in passes of up to 512 columns, so that
// one pass fills all of tensor memory (two accumulators of up to 256 columns) and the A block is fetched once
// per 512 columns of B instead of once per 256.  These kernels run at the rate shared memory is fed from L2,
// not at the tensor cores' rate: a whole pass moves 96 KB per K chunk for 256 x 512 outputs where two
// 256 x 256 tiles move 128 KB.  A ragged last pass issues a narrower second instruction (N a multiple of 32)
// instead of a whole padded tile.  D^T(m, n) is stored at out[n * out_ld + m]: consecutive lanes hold
// consecutive m, so every column of the accumulator leaves as one 128-byte warp store.
//
// Units.  Whole passes keep the traffic low but come in few, long units; so the host may cut some of the
// whole passes into their two halves of 256 columns (each a unit that uses one accumulator) where that
// evens out the pairs' loads (wide_schedule).  Units are listed longest first -- whole passes, then the ragged
// passes and the halves in the order of their cost -- and dealt to the pairs in rounds that alternate
// direction, so the pair that got the longest unit of one round gets the shortest of the next.  Within
// a class the order is batch (last to first: the kernel before went first to last), pass, M block, with
// the M block fastest (neighbouring pairs share B through L2).  A unit that needs one accumulator takes
// the two accumulators in turn, so its epilogue overlaps the next unit's contraction; after a whole pass
// the next unit starts as soon as the accumulator it needs has been read out.
// ------------------------------------------------------------------------------------------------
constexpr int kWideStages = 4;
constexpr int kWideStageBytes = 16384 + 4 * 8192;  // 128 x 64 of A + up to four 64 x 64 boxes of B per CTA
constexpr int kSmemWide = kWideStages * kWideStageBytes + 1024 + 256;
constexpr int kWideThreads = 320;  // producer, MMA, 8 epilogue warps

struct WideSchedule {
  int full_passes;   // whole passes of 512 columns per (batch, M block): n_total / 512
  int n_whole;       // whole passes kept as one unit (the first n_whole in batch / pass / M block order)
  int n_ragged;      // ragged last passes: batch * m_tiles, or 0
  int n_half;        // halves of the whole passes that were cut: 2 * (batch * m_tiles * full_passes - n_whole)
  int ragged_first;  // the ragged passes are dealt before the halves (they cost more)
  int num_units, pairs;
};

struct TnWideParams {
  int batch, m_tiles;
  WideSchedule sch;
  int num_k;      // K chunks of 64
  int n_total;    // columns of B that exist in D^T (rows of the stored matrix)
  float *out;     // D^T(j, m, n) -> out[j * out_batch + n * out_ld + m]
  size_t out_batch;
  int out_ld;
  int *status;
  HeadSlots side;  // MLP: the head kernel's slots are added up by the epilogue warps while the first operands arrive
};

// Widths of the two instructions of pass `pass` (multiples of 32; w1 may be 0).
__host__ __device__ inline void wide_pass_widths(int n_total, int pass, int *w0, int *w1) {
  const int rem = n_total - pass * 512;
  const int r32 = (rem + 31) / 32 * 32;
  *w0 = r32 < 256 ? r32 : 256;
  const int r1 = r32 - 256;
  *w1 = r1 <= 0 ? 0 : (r1 < 256 ? r1 : 256);
}

// Unit u of the list: batch j, M block mt, and up to two column ranges [c, c + w) of B (w1 = 0: one range,
// one accumulator).
struct WideUnit {
  int j, mt, c0, w0, c1, w1;
};
__host__ __device__ inline WideUnit wide_unit(int batch, int m_tiles, int n_total, const WideSchedule &s, int u) {
  const int start_ragged = s.ragged_first ? s.n_whole : s.n_whole + s.n_half;
  const int start_half = s.ragged_first ? s.n_whole + s.n_ragged : s.n_whole;
  int jr, mt, pass, half = -1;
  if (u >= start_ragged && u < start_ragged + s.n_ragged) {
    const int r = u - start_ragged;
    jr = r / m_tiles; mt = r % m_tiles; pass = s.full_passes;
  } else {
    int f = u;
    if (u >= s.n_whole) {
      const int v = u - start_half;
      f = s.n_whole + (v >> 1);
      half = v & 1;
    }
    const int per_batch = m_tiles * s.full_passes;
    jr = f / per_batch; mt = (f % per_batch) % m_tiles; pass = (f % per_batch) / m_tiles;
  }
  WideUnit q;
  q.j = batch - 1 - jr; q.mt = mt;
  wide_pass_widths(n_total, pass, &q.w0, &q.w1);
  q.c0 = pass * 512; q.c1 = q.c0 + 256;
  if (half == 0) {
    q.w1 = 0;
  } else if (half == 1) {
    q.c0 = q.c1; q.w0 = q.w1; q.w1 = 0;
  }
  return q;
}
// The i-th unit of pair `pair` (rounds alternate direction); >= num_units: none in this round.
__host__ __device__ inline int wide_unit_of(int round, int pair, int pairs) {
  return round * pairs + ((round & 1) ? pairs - 1 - pair : pair);
}

__global__ void __launch_bounds__(kWideThreads, 1)
tn_wide_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const TnWideParams p) {
  pdl_sync();
  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = smem_u32(smem_raw);
  unsigned char *tiles = smem_raw + ((1024u - (sbase & 1023u)) & 1023u);
  uint64_t *bars = reinterpret_cast<uint64_t *>(tiles + kWideStages * kWideStageBytes);
  const BarArray full{smem_u32(&bars[0])}, empty{smem_u32(&bars[kWideStages])};
  const BarArray tfull{smem_u32(&bars[2 * kWideStages])}, tempty{smem_u32(&bars[2 * kWideStages + 2])};  // per accumulator
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(&bars[2 * kWideStages + 4]);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kWideStages; ++i) {
      mbar_init(full[i], 1);
      mbar_init(empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(tfull[i], 1);
      mbar_init(tempty[i], 2 * (kWideThreads - 64));
    }
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything is signalled on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool failed = false;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int rounds = (p.sch.num_units + n_pairs - 1) / n_pairs;

  if (warp == 0) {
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      const uint64_t stream_once = l2_evict_first_policy();  // both operands are read once by this kernel
      for (int r = 0; r < rounds && !failed; ++r) {
        const int u = wide_unit_of(r, pair_id, n_pairs);
        if (u >= p.sch.num_units) continue;
        const WideUnit q = wide_unit(p.batch, p.m_tiles, p.n_total, p.sch, u);
        const int nb0 = (q.w0 / 2 + 63) / 64, nb1 = (q.w1 / 2 + 63) / 64;  // 64-column boxes of B this CTA loads
        const int m0 = q.mt * 256 + (int)rank * 128;
        const int c0 = q.c0 + (int)rank * (q.w0 / 2), c1 = q.c1 + (int)rank * (q.w1 / 2);
        const uint32_t tx = 2u * (16384u + (uint32_t)(nb0 + nb1) * 8192u);  // both CTAs signal the leader's barrier
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait(empty[st], ph ^ 1u)) { failed = true; break; }
          if (rank == 0) mbar_expect_tx(full[st], tx);
          const uint32_t a = smem_u32(tiles + st * kWideStageBytes);
          const uint32_t bar = map_to_rank(full[st], 0);
          tma_load_3d_pair_hint(a, &tmA, m0, kc * 64, q.j, bar, stream_once);
          tma_load_3d_pair_hint(a + 8192, &tmA, m0 + 64, kc * 64, q.j, bar, stream_once);
          for (int b = 0; b < nb0; ++b)
            tma_load_3d_pair_hint(a + 16384 + b * 8192, &tmB, c0 + b * 64, kc * 64, q.j, bar, stream_once);
          for (int b = 0; b < nb1; ++b)
            tma_load_3d_pair_hint(a + 16384 + (nb0 + b) * 8192, &tmB, c1 + b * 64, kc * 64, q.j, bar, stream_once);
          if (++st == kWideStages) { st = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0) {  // all 32 lanes walk the loop (uniform operands); one elected lane issues
      int st = 0, singles = 0;
      uint32_t ph = 0, eph[2] = {0u, 0u};
      for (int r = 0; r < rounds && !failed; ++r) {
        const int u = wide_unit_of(r, pair_id, n_pairs);
        if (u >= p.sch.num_units) continue;
        const WideUnit q = wide_unit(p.batch, p.m_tiles, p.n_total, p.sch, u);
        const bool both = q.w1 != 0;
        const int a0 = both ? 0 : (singles++ & 1);  // a unit of one accumulator takes them in turn
        const int nb0 = (q.w0 / 2 + 63) / 64;
        const uint32_t idesc0 = instr_desc_bf16(256, q.w0, 1, 1), idesc1 = instr_desc_bf16(256, both ? q.w1 : 32, 1, 1);
        const uint32_t acc0 = tmem_base + (uint32_t)a0 * 256u, acc1 = tmem_base + 256u;
        if (!mbar_wait_warp(tempty[a0], (a0 ? eph[1] : eph[0]) ^ 1u)) { failed = true; break; }
        if (both && !mbar_wait_warp(tempty[1], eph[1] ^ 1u)) { failed = true; break; }
        tc_fence_after();
        for (int kc = 0; kc < p.num_k; ++kc) {
          if (!mbar_wait_warp(full[st], ph)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a = smem_u32(tiles + st * kWideStageBytes);
          // M/N-major: 64-element boxes 8192 B apart, 8-row K groups 1024 B apart
          const uint64_t ad = smem_desc_sw128(a, 8192, 1024), bd0 = smem_desc_sw128(a + 16384, 8192, 1024),
                         bd1 = smem_desc_sw128(a + 16384 + nb0 * 8192, 8192, 1024);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) {  // 16 rows of K = 2048 bytes per instruction
            mma_bf16_pair(acc0, ad + (uint64_t)(k4 * 128), bd0 + (uint64_t)(k4 * 128), idesc0, (kc | k4) != 0);
            if (both)
              mma_bf16_pair(acc1, ad + (uint64_t)(k4 * 128), bd1 + (uint64_t)(k4 * 128), idesc1, (kc | k4) != 0);
          }
          mma_commit_pair(empty[st], 3);
          if (++st == kWideStages) { st = 0; ph ^= 1u; }
        }
        if (failed) break;
        mma_commit_pair(tfull[a0], 3);
        if (both) mma_commit_pair(tfull[1], 3);
        if (a0 || both) eph[1] ^= 1u;
        if (!a0) eph[0] ^= 1u;
      }
    }
  } else {
    const int q4 = warp & 3, half = (warp - 2) >> 2;  // warps w and w + 4 share a quadrant and alternate 32-column chunks
    if (p.side.slots) {
      const long long total = (long long)p.side.k * p.side.wstride, nthr = (long long)gridDim.x * (kWideThreads - 64);
      for (long long e = (long long)blockIdx.x * (kWideThreads - 64) + ((int)threadIdx.x - 64); e < total; e += nthr)
        head_reduce_one(p.side, (int)(e / p.side.wstride), (int)(e % p.side.wstride));
    }
    int singles = 0;
    uint32_t fph[2] = {0u, 0u};
    for (int r = 0; r < rounds && !failed; ++r) {
      const int u = wide_unit_of(r, pair_id, n_pairs);
      if (u >= p.sch.num_units) continue;
      const WideUnit q = wide_unit(p.batch, p.m_tiles, p.n_total, p.sch, u);
      const bool both = q.w1 != 0;
      const int a0 = both ? 0 : (singles++ & 1);
      const int m = q.mt * 256 + (int)rank * 128 + q4 * 32 + lane;
      float *dst = p.out + (size_t)q.j * p.out_batch + m;
      for (int x = 0; x < (both ? 2 : 1); ++x) {
        const int acc = both ? x : a0, w = x ? q.w1 : q.w0, c = x ? q.c1 : q.c0;
        if (!mbar_wait(tfull[acc], acc ? fph[1] : fph[0])) { failed = true; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)acc * 256u;
        for (int ch = half; ch < (w >> 5); ch += 2) {
          const int n0 = c + ch * 32;
          if (n0 >= p.n_total) continue;  // (uniform per warp)
          float v[32];
          tmem_ld32(taddr + (uint32_t)(ch * 32), v);
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (n0 + i < p.n_total) dst[(size_t)(n0 + i) * p.out_ld] = v[i];
        }
        tc_fence_before();
        mbar_arrive_cluster(map_to_rank(tempty[acc], 0));
        if (acc) fph[1] ^= 1u; else fph[0] ^= 1u;
      }
    }
  }
  pair_teardown(warp, tmem_base, failed, p.status);
}

// Which whole passes to cut in halves.  Cost of a unit per K chunk, in SM cycles: the slower of feeding shared
// memory (measured: about 41 bytes per cycle and SM in these kernels) and the tensor cores (a 256 x w x 16
// instruction takes w / 2 cycles), plus reading the accumulators out.  Candidates: keep all whole passes, or
// cut the last t of them, t up to two rounds of pairs; each is dealt as the kernel deals and the one with
// the shortest longest pair wins (ties: fewer cuts, i.e. less traffic).
static double wide_unit_cost(int w0, int w1, int num_k) {
  const int nb = (w0 / 2 + 63) / 64 + (w1 / 2 + 63) / 64;
  const double fill = (16384.0 + 8192.0 * nb) / 41.0, mma = 2.0 * (w0 + w1);
  return (fill > mma ? fill : mma) * num_k + 20.0 * (w0 + w1);
}
static WideSchedule wide_schedule(int batch, int m_tiles, int n_total, int num_k, int max_pairs) {
  WideSchedule s;
  s.full_passes = n_total / 512;
  const int whole = batch * m_tiles * s.full_passes;
  int rw0 = 0, rw1 = 0;
  if (n_total % 512) wide_pass_widths(n_total, s.full_passes, &rw0, &rw1);
  s.n_ragged = (n_total % 512) ? batch * m_tiles : 0;
  const double c_whole = wide_unit_cost(256, 256, num_k), c_half = wide_unit_cost(256, 0, num_k),
               c_ragged = s.n_ragged ? wide_unit_cost(rw0, rw1, num_k) : 0.0;
  s.ragged_first = c_ragged >= c_half ? 1 : 0;
  WideSchedule best = s;
  double best_span = -1.0;
  std::vector<double> load;
  const int t_max = whole < 2 * max_pairs ? whole : 2 * max_pairs;
  for (int t = 0; t <= t_max; ++t) {
    s.n_whole = whole - t;
    s.n_half = 2 * t;
    s.num_units = s.n_whole + s.n_ragged + s.n_half;
    s.pairs = s.num_units < max_pairs ? s.num_units : max_pairs;
    if (s.pairs < 1) s.pairs = 1;
    load.assign(s.pairs, 0.0);
    const int second = s.ragged_first ? s.n_ragged : s.n_half;
    for (int u = 0; u < s.num_units; ++u) {
      const int r = u / s.pairs, pos = u % s.pairs, pair = (r & 1) ? s.pairs - 1 - pos : pos;
      const double c = u < s.n_whole ? c_whole
                       : (u < s.n_whole + second ? (s.ragged_first ? c_ragged : c_half)
                                                 : (s.ragged_first ? c_half : c_ragged));
      load[pair] += c;
    }
    double span = 0.0;
    for (double v : load) span = v > span ? v : span;
    if (best_span < 0.0 || span < best_span * (1.0 - 1e-9)) {
      best_span = span;
      best = s;
    }
  }
  return best;
}

// The opt-in shared-memory size of a kernel is set once per device and kernel, not on every launch.
struct SmemAttrDone {
  const void *kern;
  int dev, bytes;
};
template <typename Kern>
cudaError_t ensure_smem_attr(Kern kern, int smem_bytes) {
  static std::mutex mu;
  static std::vector<SmemAttrDone> done;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const void *key = reinterpret_cast<const void *>(kern);  // kernels of one signature share this template instance
  std::lock_guard<std::mutex> lock(mu);
  for (auto &d : done)
    if (d.kern == key && d.dev == dev) {
      if (d.bytes >= smem_bytes) return cudaSuccess;
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
      if (e == cudaSuccess) d.bytes = smem_bytes;
      return e;
    }
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e == cudaSuccess) done.push_back({key, dev, smem_bytes});
  return e;
}

// Launch on clusters of two CTAs.
template <typename Kern, typename Params>
cudaError_t launch_pair(Kern kern, int threads, int pair_tiles, int sms, const CUtensorMap &m0, const CUtensorMap &m1,
                        const Params &p, cudaStream_t stream, int smem_bytes = kSmemPair) {
  cudaError_t e = ensure_smem_attr(kern, smem_bytes);
  if (e != cudaSuccess) return e;
  int pairs = sms / 2;
  if (pair_tiles < pairs) pairs = pair_tiles;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kern, m0, m1, p);
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

inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }

// Largest number of CTAs of the head kernel whose contiguous tile ranges touch one partition.
int head_max_slots(int k, int tpp, int grid) {
  int worst = 1;
  for (int j = 0; j < k; ++j) {
    // first and last CTA whose range [begin(c), begin(c + 1)) meets the tiles [j tpp, (j + 1) tpp) of partition j
    const int cfirst = (int)(((long long)(j * tpp + 1) * grid - 1) / ((long long)k * tpp));
    const int clast = (int)(((long long)((j + 1) * tpp) * grid - 1) / ((long long)k * tpp));
    if (clast - cfirst + 1 > worst) worst = clast - cfirst + 1;
  }
  return worst;
}

int head_grid(int k, int rows, int sms) {
  const int tiles = k * ((rows + 127) / 128);
  return tiles < sms ? tiles : (sms > 0 ? sms : 1);
}

}  // namespace

// What the dense launchers keep between calls, per plan: the tensor maps and derived sizes of the last
// softmax and MLP problem (encoding 5-9 maps and walking the head kernel's tile ranges on every call is host
// time on the critical path of a caller that synchronises per step), and the data prepared once.
struct DenseState {
  struct {
    bool valid = false;
    int k = 0, rows = 0, d = 0, C = 0, sms = 0;
    const void *X = nullptr, *scratch = nullptr;
    CUtensorMap tmXa, tmXb, tmW, tmWh, tmR;
    WideSchedule wide;  // units of the backward contraction (CTA-pair path)
  } sm;
  struct {
    bool valid = false;
    int k = 0, rows = 0, d = 0, hidden = 0, C = 0, sms = 0;
    const void *Xb = nullptr, *scratch = nullptr;
    int max_slots = 0;
    CUtensorMap tmXa, tmXb, tmW, tmWh, tmH, tmHa, tmD1, tmD1s, tmD2, tmW2t, tmW2k;
    WideSchedule wide;  // units of the [dW1; db1] contraction (CTA-pair path)
  } mlp;
  // bf16 copy [X 1] of an MLP's data matrix made by prepare_mlp_data (owned here)
  __nv_bfloat16 *Xb_prep = nullptr;
  size_t Xb_prep_bytes = 0;
  const void *prep_src = nullptr;
  int prep_k = 0, prep_rows = 0, prep_d = 0;
};

// The unit list of the wide backward contraction as the kernel walks it, for inspection: row u of `units`
// gets {pair, round, batch j, M block, c0, w0, c1, w1}.  Returns the number of units (rows written: at most cap).
int wide_schedule_units(int batch, int m_tiles, int n_total, int num_k, int max_pairs, int *units, int cap,
                        int *pairs_out) {
  const WideSchedule s = wide_schedule(batch, m_tiles, n_total, num_k, max_pairs);
  if (pairs_out) *pairs_out = s.pairs;
  const int rounds = (s.num_units + s.pairs - 1) / s.pairs;
  int n = 0;
  for (int r = 0; r < rounds; ++r)
    for (int pair = 0; pair < s.pairs; ++pair) {
      const int u = wide_unit_of(r, pair, s.pairs);
      if (u >= s.num_units) continue;
      if (n < cap) {
        const WideUnit q = wide_unit(batch, m_tiles, n_total, s, u);
        int *row = units + (size_t)n * 8;
        row[0] = pair; row[1] = r; row[2] = q.j; row[3] = q.mt; row[4] = q.c0; row[5] = q.w0; row[6] = q.c1; row[7] = q.w1;
      }
      ++n;
    }
  return n;
}

void dense_state_free(DenseState *st) {
  if (!st) return;
  if (st->Xb_prep) cudaFree(st->Xb_prep);
  delete st;
}

size_t dense_state_bytes(const DenseState *st) { return st ? st->Xb_prep_bytes : 0; }

static DenseState *state_of(DenseState **slot) {
  if (!*slot) *slot = new (std::nothrow) DenseState();
  return *slot;
}

size_t softmax_scratch_bytes(int k, int rows, int d, int C) {
  const size_t wt = ((size_t)C * d * 2 + 255) / 256 * 256;
  const size_t r = ((size_t)k * rows * C * 2 + 255) / 256 * 256;
  const size_t g = (size_t)k * d * C * 4;
  return wt + r + g;
}

cudaError_t launch_softmax_grad(int k, int rows, int d, int C, const void *X, const int *y, const float *W,
                                unsigned char *scratch, float **G_out, int *status, int sms, cudaStream_t stream,
                                DenseState **state) {
  if (C % 16 != 0 || C < 16 || C > 256 || d % 8 != 0 || d < 8) return cudaErrorInvalidValue;
  DenseState *st = state_of(state);
  if (!st) return cudaErrorMemoryAllocation;
  const size_t wt_bytes = ((size_t)C * d * 2 + 255) / 256 * 256;
  const size_t r_bytes = ((size_t)k * rows * C * 2 + 255) / 256 * 256;
  __nv_bfloat16 *Wt = reinterpret_cast<__nv_bfloat16 *>(scratch);
  __nv_bfloat16 *R = reinterpret_cast<__nv_bfloat16 *>(scratch + wt_bytes);
  float *G = reinterpret_cast<float *>(scratch + wt_bytes + r_bytes);
  *G_out = G;

  auto &c = st->sm;
  if (!(c.valid && c.k == k && c.rows == rows && c.d == d && c.C == C && c.sms == sms && c.X == X &&
        c.scratch == scratch)) {
    c.valid = false;
    const uint64_t xdims[3] = {(uint64_t)d, (uint64_t)rows, (uint64_t)k};
    const uint32_t xbox_a[3] = {64, 128, 1}, xbox_b[3] = {64, 64, 1};
    const uint64_t wdims[2] = {(uint64_t)d, (uint64_t)C};
    const uint32_t wbox[2] = {64, 256}, wbox_h[2] = {64, 128};  // whole tile / half of the class rows per CTA of a pair
    const uint64_t rdims[3] = {(uint64_t)C, (uint64_t)rows, (uint64_t)k};
    const uint32_t rbox[3] = {64, 64, 1};
    if (!make_map(&c.tmXa, X, 3, xdims, xbox_a) || !make_map(&c.tmXb, X, 3, xdims, xbox_b) ||
        !make_map(&c.tmW, Wt, 2, wdims, wbox) || !make_map(&c.tmWh, Wt, 2, wdims, wbox_h) ||
        !make_map(&c.tmR, R, 3, rdims, rbox))
      return cudaErrorInvalidValue;
    if (C == 256 && sms >= 2) c.wide = wide_schedule(k, 1, d, (rows + 63) / 64, sms / 2);
    c.k = k; c.rows = rows; c.d = d; c.C = C; c.sms = sms; c.X = X; c.scratch = scratch;
    c.valid = true;
  }

  dim3 tg((C + 31) / 32, (d + 31) / 32);
  launch_k(transpose_to_bf16_kernel, tg, 256, 0, stream, W, nullptr, Wt, d, C, d);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  const bool pair = (C == 256) && sms >= 2;
  FwdParams p;
  p.rows = rows; p.n_total = C; p.n_tiles = 1;
  p.num_k = (d + 63) / 64;
  p.y = y; p.out = R; p.out_ld = C; p.ones_col = -1; p.status = status;
  if (pair) {
    p.row_blocks = (rows + 255) / 256;
    p.num_tiles = k * p.row_blocks;
    e = launch_pair(fwd_pair_kernel<0>, kFwdThreads, p.num_tiles, sms, c.tmXa, c.tmWh, p, stream);
  } else {
    if ((e = ensure_smem_attr(fwd_kernel<0>, kSmemFwd)) != cudaSuccess) return e;
    p.row_blocks = (rows + 127) / 128;
    p.num_tiles = k * p.row_blocks;
    launch_k(fwd_kernel<0>, p.num_tiles < sms ? p.num_tiles : sms, kFwdThreads, kSmemFwd, stream, c.tmXa, c.tmW, p);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) return e;

  if (pair) {
    // G_j^T = R_j^T X_j: the residual (C = 256 classes) on the M side, the data matrix on the N side in passes of
    // 512 features; the transposed store puts element (class, feature) at G[feature][class]
    TnWideParams wp;
    wp.batch = k; wp.m_tiles = 1; wp.sch = c.wide; wp.num_k = (rows + 63) / 64;
    wp.n_total = d; wp.out = G; wp.out_batch = (size_t)d * C; wp.out_ld = C; wp.status = status;
    wp.side = HeadSlots{};
    return launch_pair(tn_wide_pair_kernel, kWideThreads, wp.sch.num_units, sms, c.tmR, c.tmXb, wp, stream, kSmemWide);
  }
  TnParams t;
  t.batch = k; t.n_tiles = 1;
  t.num_k = (rows + 63) / 64;
  t.N = C; t.nbox = (C + 63) / 64;
  t.m_store = d; t.n_store = C;
  t.out = G; t.out_batch = (size_t)d * C; t.out_ld = C;
  t.status = status;
  if ((e = ensure_smem_attr(tn_gemm_kernel, kSmemTc)) != cudaSuccess) return e;
  t.m_tiles = (d + 127) / 128; t.num_tiles = k * t.m_tiles;
  launch_k(tn_gemm_kernel, t.num_tiles < sms ? t.num_tiles : sms, kTcThreads, kSmemTc, stream, c.tmXb, c.tmR, t);
  return cudaGetLastError();
}

size_t mlp_scratch_bytes(int k, int rows, int d, int hidden, int C) {
  const size_t dpad = (size_t)(d + 1 + 7) / 8 * 8, hpad = (size_t)(hidden + 1 + 7) / 8 * 8;
  const size_t l = (size_t)d * hidden + hidden + (size_t)hidden * C + C, lpad = (l + 3) / 4 * 4;
  const size_t kr = (size_t)k * rows;
  const int slots = head_max_slots(k, (rows + 127) / 128, head_grid(k, rows, device_sm_count()));
  return up256(kr * dpad * 2) + up256((size_t)hidden * dpad * 2) + up256(kr * hpad * 2) + up256(kr * hidden * 2) +
         up256(kr * 64 * 2) + up256((size_t)16 * hidden * 2) + up256((size_t)hidden * 64 * 2) +
         up256((size_t)k * slots * ((size_t)hidden * C + C) * 4) + up256((size_t)k * lpad * 4);
}

int mlp_launch_count(int hidden) {
  // operand preparation, forward, head, dW1, encode; dW2 by a contraction of its own or by the head kernel plus a
  // sum over its slots, which the wide backward kernel (hidden a multiple of 256) does on the side
  return hidden % 256 == 0 ? 5 : 6;
}

// bf16 copy [X 1] of the data matrix of an MLP, made once: the data is assigned to the workers before
// training starts (Section II-C) and does not change from iteration to iteration, so the conversion the
// tensor cores need (fp32 -> bf16, plus the column of ones that carries the bias) is no part of a step.
// X == nullptr drops the copy.
cudaError_t prepare_mlp_data(DenseState **state, int k, int rows, int d, const float *X, cudaStream_t stream) {
  DenseState *st = state_of(state);
  if (!st) return cudaErrorMemoryAllocation;
  st->prep_src = nullptr;
  st->mlp.valid = false;
  if (!X) {
    if (st->Xb_prep) {
      cudaError_t e = cudaDeviceSynchronize();
      if (e != cudaSuccess) return e;
      cudaFree(st->Xb_prep);
      st->Xb_prep = nullptr;
      st->Xb_prep_bytes = 0;
    }
    return cudaSuccess;
  }
  if (d % 8 != 0 || k < 1 || rows < 1) return cudaErrorInvalidValue;
  const int dpad = (d + 1 + 7) / 8 * 8;
  const size_t kr = (size_t)k * rows, bytes = up256(kr * dpad * 2);
  if (bytes > st->Xb_prep_bytes) {
    if (st->Xb_prep) {
      cudaError_t e = cudaDeviceSynchronize();
      if (e != cudaSuccess) return e;
      cudaFree(st->Xb_prep);
      st->Xb_prep = nullptr;
      st->Xb_prep_bytes = 0;
    }
    cudaError_t e = cudaMalloc(&st->Xb_prep, bytes);
    if (e != cudaSuccess) return e;
    st->Xb_prep_bytes = bytes;
  }
  MlpPrepParams pp = {};
  pp.X = X; pp.Xb = st->Xb_prep; pp.rows_total = (long long)kr; pp.d = d; pp.dpad = dpad;
  pp.tr_bx = 1; pp.tr_blocks = 0; pp.w2_blocks = 0;
  const long long groups = (long long)kr * (dpad / 8);
  launch_k(mlp_prep_kernel, (unsigned)((groups + 255) / 256), 256, 0, stream, pp);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  st->prep_src = X; st->prep_k = k; st->prep_rows = rows; st->prep_d = d;
  return cudaSuccess;
}

cudaError_t launch_mlp_grad(int k, int rows, int d, int hidden, int C, const float *X, const int *y, const float *theta,
                            unsigned char *scratch, float **G_out, long long *G_ld, int *status, int sms,
                            cudaStream_t stream, DenseState **state) {
  if (d % 8 != 0 || hidden % 16 != 0 || hidden < 16 || hidden > 512 || (hidden > 256 && hidden % 256 != 0) || C < 1 ||
      C > 16)
    return cudaErrorInvalidValue;
  DenseState *st = state_of(state);
  if (!st) return cudaErrorMemoryAllocation;
  const int dpad = (d + 1 + 7) / 8 * 8, hpad = (hidden + 1 + 7) / 8 * 8;
  const size_t l = (size_t)d * hidden + hidden + (size_t)hidden * C + C, lpad = (l + 3) / 4 * 4;
  const size_t kr = (size_t)k * rows;
  unsigned char *ptr = scratch;
  __nv_bfloat16 *Xb = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * dpad * 2);
  __nv_bfloat16 *W1t = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256((size_t)hidden * dpad * 2);
  __nv_bfloat16 *H = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * hpad * 2);
  __nv_bfloat16 *D1 = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * hidden * 2);
  __nv_bfloat16 *D2 = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256(kr * 64 * 2);
  __nv_bfloat16 *W2t = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256((size_t)16 * hidden * 2);
  __nv_bfloat16 *W2k = reinterpret_cast<__nv_bfloat16 *>(ptr); ptr += up256((size_t)hidden * 64 * 2);
  // the copy made by prepare_mlp_data for this very data matrix replaces the per-call conversion
  const bool prepared = st->Xb_prep && st->prep_src == X && st->prep_k == k && st->prep_rows == rows && st->prep_d == d;
  if (prepared) Xb = st->Xb_prep;
  const int tpp = (rows + 127) / 128, hgrid = head_grid(k, rows, sms);

  const int nchunk = hidden / 64, nhalf = (hidden + 255) / 256;
  const size_t head_tc_smem = (size_t)nchunk * 16384 + 16384 + (size_t)nhalf * 32768 + (size_t)nchunk * 2048 + 1024 + 1024;
  const bool head_tc = hidden % 64 == 0 && head_tc_smem <= 232448;
  const bool fuse_w2 = head_tc && hidden % 128 == 0;  // the head forms [dW2; db2] itself: no column of ones behind h

  auto &c = st->mlp;
  if (!(c.valid && c.k == k && c.rows == rows && c.d == d && c.hidden == hidden && c.C == C && c.sms == sms &&
        c.Xb == Xb && c.scratch == scratch)) {
    c.valid = false;
    // scratch was sized with the slot count of a grid on every SM of the device
    c.max_slots = head_max_slots(k, tpp, head_grid(k, rows, device_sm_count()));
    if (head_max_slots(k, tpp, hgrid) > c.max_slots) return cudaErrorInvalidValue;
    const uint64_t xdims[3] = {(uint64_t)dpad, (uint64_t)rows, (uint64_t)k};
    const uint32_t box_a[3] = {64, 128, 1}, box_b[3] = {64, 64, 1};
    const uint64_t wdims[2] = {(uint64_t)dpad, (uint64_t)hidden};
    const uint32_t wbox[2] = {64, 256}, wbox_h[2] = {64, 128};
    const uint64_t hdims[3] = {(uint64_t)hpad, (uint64_t)rows, (uint64_t)k};
    const uint64_t d1dims[3] = {(uint64_t)hidden, (uint64_t)rows, (uint64_t)k};
    const uint64_t d2dims[3] = {64, (uint64_t)rows, (uint64_t)k};
    // h in 128-row boxes (head: tmHa) and in 64-row boxes (backward operand: tmH); the same 128 x 64 box serves the
    // head's loads of h and its stores of delta1 (tmD1s)
    if (!make_map(&c.tmXa, Xb, 3, xdims, box_a) || !make_map(&c.tmXb, Xb, 3, xdims, box_b) ||
        !make_map(&c.tmW, W1t, 2, wdims, wbox) || !make_map(&c.tmWh, W1t, 2, wdims, wbox_h) ||
        !make_map(&c.tmH, H, 3, hdims, box_b) || !make_map(&c.tmHa, H, 3, hdims, box_a) ||
        !make_map(&c.tmD1, D1, 3, d1dims, box_b) || !make_map(&c.tmD1s, D1, 3, d1dims, box_a) ||
        !make_map(&c.tmD2, D2, 3, d2dims, box_b))
      return cudaErrorInvalidValue;
    if (head_tc) {
      const uint64_t w2tdims[2] = {(uint64_t)hidden, 16}, w2kdims[2] = {64, (uint64_t)hidden};
      const uint32_t box_w2t[2] = {64, 16}, box_w2k[2] = {64, 256};
      if (!make_map(&c.tmW2t, W2t, 2, w2tdims, box_w2t) || !make_map(&c.tmW2k, W2k, 2, w2kdims, box_w2k))
        return cudaErrorInvalidValue;
    }
    if (hidden % 256 == 0 && sms >= 2) c.wide = wide_schedule(k, hidden / 256, d + 1, (rows + 63) / 64, sms / 2);
    c.k = k; c.rows = rows; c.d = d; c.hidden = hidden; c.C = C; c.sms = sms; c.Xb = Xb; c.scratch = scratch;
    c.valid = true;
  }
  const int max_slots = c.max_slots;
  float *slots = reinterpret_cast<float *>(ptr); ptr += up256((size_t)k * max_slots * ((size_t)hidden * C + C) * 4);
  float *G = reinterpret_cast<float *>(ptr);
  *G_out = G;
  *G_ld = (long long)lpad;
  const float *W1 = theta, *b1 = theta + (size_t)d * hidden, *W2 = b1 + hidden, *b2 = W2 + (size_t)hidden * C;

  MlpPrepParams pp;
  pp.X = X; pp.Xb = Xb; pp.rows_total = prepared ? 0 : (long long)kr; pp.d = d; pp.dpad = dpad;
  pp.W1 = W1; pp.b1 = b1; pp.W1t = W1t; pp.hidden = hidden;
  pp.W2 = W2; pp.C = C; pp.W2t = W2t; pp.W2k = W2k;
  pp.tr_bx = (hidden + 31) / 32; pp.tr_blocks = pp.tr_bx * ((dpad + 31) / 32);
  pp.w2_blocks = head_tc ? (hidden * 64 + 255) / 256 : 0;
  const long long groups = pp.rows_total * (dpad / 8);
  launch_k(mlp_prep_kernel, (unsigned)(pp.tr_blocks + pp.w2_blocks + (groups + 255) / 256), 256, 0, stream, pp);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  // H = relu([X 1] [W1; b1]), with its own column of ones behind the hidden units
  FwdParams p;
  p.rows = rows; p.n_total = hidden; p.row_blocks = (rows + 127) / 128; p.n_tiles = (hidden + 255) / 256;
  p.num_tiles = k * p.row_blocks * p.n_tiles; p.num_k = (dpad + 63) / 64;
  p.y = y; p.out = H; p.out_ld = hpad; p.ones_col = fuse_w2 ? -1 : hidden; p.status = status;
  const bool pair = (hidden % 256 == 0) && sms >= 2;  // CTA pairs: 256 rows per tile, half of W1^T per CTA
  if (pair) {
    p.row_blocks = (rows + 255) / 256;
    p.num_tiles = k * p.row_blocks * p.n_tiles;
    e = launch_pair(fwd_pair_kernel<1>, kFwdThreads, p.num_tiles, sms, c.tmXa, c.tmWh, p, stream);
  } else {
    if ((e = ensure_smem_attr(fwd_kernel<1>, kSmemFwd)) != cudaSuccess) return e;
    launch_k(fwd_kernel<1>, p.num_tiles < sms ? p.num_tiles : sms, kFwdThreads, kSmemFwd, stream, c.tmXa, c.tmW, p);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) return e;

  HeadSlots head_slots = {};
  if (head_tc) {
    HeadTcParams hp;
    hp.hidden = hidden; hp.C = C; hp.rows = rows; hp.tiles_per_part = tpp; hp.num_tiles = k * tpp;
    hp.b2 = b2; hp.y = y; hp.D2 = D2; hp.fuse = fuse_w2 ? 1 : 0;
    hp.slots = slots; hp.max_slots = max_slots; hp.status = status;
    if ((e = ensure_smem_attr(mlp_head_tc_kernel, (int)head_tc_smem)) != cudaSuccess) return e;
    launch_k(mlp_head_tc_kernel, hgrid, kHeadTcThreads, head_tc_smem, stream, c.tmHa, c.tmW2t, c.tmW2k, c.tmD1s, hp);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (fuse_w2) {
      head_slots.slots = slots; head_slots.max_slots = max_slots; head_slots.wstride = hidden * C + C;
      head_slots.tpp = tpp; head_slots.num_tiles = k * tpp; head_slots.grid = hgrid; head_slots.k = k;
      head_slots.G = G + (size_t)d * hidden + hidden; head_slots.g_batch = lpad;
      if (!pair) {  // (the wide backward kernel below adds the slots up on the side)
        launch_k(head_reduce_kernel, dim3((head_slots.wstride + 255) / 256, k), 256, 0, stream, head_slots);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
      }
    }
  } else {
    const int cpad = (C + 3) / 4 * 4;
    const size_t head_smem = ((size_t)hidden * cpad + cpad + 4 * kHeadRows * cpad) * sizeof(float) + (size_t)kHeadRows * hpad * 2;
    const unsigned head_blocks = (unsigned)((kr + kHeadRows - 1) / kHeadRows);
#define NGC_LAUNCH_HEAD(CP)                                                                                       \
  do {                                                                                                            \
    e = ensure_smem_attr(mlp_head_kernel<CP>, (int)head_smem);                                                    \
    if (e != cudaSuccess) return e;                                                                               \
    launch_k(mlp_head_kernel<CP>, head_blocks, kHeadThreads, head_smem, stream, H, hpad, hidden, C, W2, b2, y,          \
                                                                          (long long)kr, D1, D2);                 \
  } while (0)
    if (cpad == 4) NGC_LAUNCH_HEAD(4);
    else if (cpad == 8) NGC_LAUNCH_HEAD(8);
    else if (cpad == 12) NGC_LAUNCH_HEAD(12);
    else NGC_LAUNCH_HEAD(16);
#undef NGC_LAUNCH_HEAD
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }

  TnParams t;
  t.batch = k; t.status = status; t.num_k = (rows + 63) / 64;
  // [dW1; db1] = [X 1]^T delta1
  t.m_tiles = (d + 1 + 127) / 128; t.n_tiles = (hidden + 255) / 256; t.num_tiles = k * t.m_tiles * t.n_tiles;
  t.N = hidden < 256 ? hidden : 256; t.nbox = (t.N + 63) / 64;
  t.m_store = d + 1; t.n_store = t.N;
  t.out = G; t.out_batch = lpad; t.out_ld = hidden;
  if (pair) {
    // delta1 on the M side (hidden is a multiple of 256), [X 1] on the N side in passes of 512 columns
    TnWideParams wp;
    wp.batch = k; wp.m_tiles = hidden / 256; wp.sch = c.wide; wp.num_k = (rows + 63) / 64;
    wp.n_total = d + 1; wp.out = G; wp.out_batch = lpad; wp.out_ld = hidden; wp.status = status;
    wp.side = head_slots;
    e = launch_pair(tn_wide_pair_kernel, kWideThreads, wp.sch.num_units, sms, c.tmD1, c.tmXb, wp, stream, kSmemWide);
  } else {
    if ((e = ensure_smem_attr(tn_gemm_kernel, kSmemTc)) != cudaSuccess) return e;
    launch_k(tn_gemm_kernel, t.num_tiles < sms ? t.num_tiles : sms, kTcThreads, kSmemTc, stream, c.tmXb, c.tmD1, t);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess || fuse_w2) return e;
  // [dW2; db2] = [h 1]^T delta2
  if ((e = ensure_smem_attr(tn_gemm_kernel, kSmemTc)) != cudaSuccess) return e;
  t.m_tiles = (hidden + 1 + 127) / 128; t.n_tiles = 1; t.num_tiles = k * t.m_tiles;
  t.N = 16; t.nbox = 1;
  t.m_store = hidden + 1; t.n_store = C;
  t.out = G + (size_t)d * hidden + hidden; t.out_batch = lpad; t.out_ld = C;
  launch_k(tn_gemm_kernel, t.num_tiles < sms ? t.num_tiles : sms, kTcThreads, kSmemTc, stream, c.tmH, c.tmD2, t);
  return cudaGetLastError();
}

}  // namespace ngc
