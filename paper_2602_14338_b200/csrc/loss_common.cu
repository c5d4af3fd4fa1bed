// Host-launched helpers of stage (b): the row-tile work list over runs of kept
// rollouts and the fixed-order reduction of the loss partials.
#include "loss_common.cuh"

namespace {

// Inclusive block scan (1024 threads) with a generic associative operator.
template <typename T, typename Op>
__device__ T block_scan_incl(T v, Op op, T identity, T* s_warp) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const T u = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v = op(u, v);
  }
  if (lane == 31) s_warp[wid] = v;
  __syncthreads();
  if (wid == 0) {
    T x = s_warp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const T u = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x = op(u, x);
    }
    s_warp[lane] = x;
  }
  __syncthreads();
  const T prefix = wid > 0 ? s_warp[wid - 1] : identity;
  v = op(prefix, v);
  __syncthreads();
  return v;
}

struct MaxOp { __device__ int operator()(int a, int b) const { return a > b ? a : b; } };
struct AddOp { __device__ int operator()(int a, int b) const { return a + b; } };

// A tile is tile_rows consecutive token rows starting at a row of a kept rollout.  Tiles
// are laid from the first row of each maximal run of consecutive kept rollouts, so rows
// past the end of a run (which belong to a dropped rollout, or lie beyond T) are the
// only rows a tile covers without need.  Rollout i owns the tiles that start inside it.
__global__ void __launch_bounds__(1024) build_tiles_kernel(long long T, int R, const int64_t* __restrict__ cs,
                                                           const uint8_t* __restrict__ keep, int tile_rows,
                                                           int32_t* __restrict__ tile_row, int32_t* __restrict__ tile_valid,
                                                           int32_t* __restrict__ n_tiles, int max_tiles) {
  __shared__ int s_warp[32];
  int carry_start = -1;   // index of the rollout that starts the current run (if the previous rollout is kept)
  int carry_tiles = 0;
  for (int base = 0; base < R; base += 1024) {
    const int i = base + threadIdx.x;
    bool kp = false;
    long long a = 0, b = 0;
    if (i < R) {
      a = cs[i]; b = cs[i + 1];
      kp = keep[i] != 0 && a >= 0 && b > a && b <= T;
    }
    const bool prev_kp = (i > 0 && i < R) ? (keep[i - 1] != 0 && cs[i - 1] >= 0 && cs[i] > cs[i - 1] && cs[i] <= T) : false;
    // run start of rollout i: the latest run-starting rollout at or before i
    int start_mark = (kp && !prev_kp) ? i : -1;
    int run_start = block_scan_incl<int>(start_mark, MaxOp(), -1, s_warp);
    if (run_start < 0) run_start = carry_start;
    int cnt = 0;
    long long first_k = 0, s0 = 0;
    if (kp && run_start >= 0) {
      s0 = cs[run_start];
      first_k = (a - s0 + tile_rows - 1) / tile_rows;
      const long long end_k = (b - s0 + tile_rows - 1) / tile_rows;
      cnt = (int)(end_k - first_k);
    }
    const int incl = block_scan_incl<int>(cnt, AddOp(), 0, s_warp);
    const int off = carry_tiles + incl - cnt;
    for (int k = 0; k < cnt; ++k) {
      if (off + k >= max_tiles) break;
      const long long start = s0 + (first_k + k) * tile_rows;
      // rows of the tile that still belong to this run: walk over the kept rollouts that follow
      int j = i;
      long long end = b;
      while (end < start + tile_rows && j + 1 < R && keep[j + 1] != 0 && cs[j + 2] > cs[j + 1] && cs[j + 2] <= T) {
        ++j;
        end = cs[j + 1];
      }
      const long long valid = end - start < tile_rows ? end - start : tile_rows;
      tile_row[off + k] = (int32_t)start;
      tile_valid[off + k] = (int32_t)valid;
    }
    // carry to the next chunk of rollouts
    __shared__ int s_carry[2];
    __syncthreads();
    if (threadIdx.x == 1023) {
      s_carry[0] = kp ? run_start : -1;
      s_carry[1] = carry_tiles + incl;
    }
    __syncthreads();
    carry_start = s_carry[0];
    carry_tiles = s_carry[1];
    __syncthreads();
  }
  if (threadIdx.x == 0) *n_tiles = carry_tiles < max_tiles ? carry_tiles : max_tiles;
}

__global__ void __launch_bounds__(256) dense_tiles_kernel(long long T, int tile_rows, int32_t* __restrict__ tile_row,
                                                          int32_t* __restrict__ tile_valid, int32_t* __restrict__ n_tiles,
                                                          int max_tiles) {
  const long long n = (T + tile_rows - 1) / tile_rows;
  const int count = (int)(n < max_tiles ? n : max_tiles);
  for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < count; k += gridDim.x * blockDim.x) {
    const long long start = (long long)k * tile_rows;
    tile_row[k] = (int32_t)start;
    tile_valid[k] = (int32_t)(T - start < tile_rows ? T - start : tile_rows);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *n_tiles = count;
}

// Sum n partial records of `stride` doubles each in a fixed order: thread j adds records
// j, j+1024, ... in increasing order, then a fixed shuffle/shared tree combines threads.
__global__ void __launch_bounds__(1024) finalize_kernel(const double* __restrict__ part, int n, int stride,
                                                        float* loss, float* metrics, int accumulate) {
  __shared__ double s[32][kPartialStride];
  double acc[kPartialStride];
  for (int k = 0; k < kPartialStride; ++k) acc[k] = 0.0;
  for (int r = threadIdx.x; r < n; r += 1024)
    for (int k = 0; k < kPartialStride; ++k) acc[k] += part[(size_t)r * stride + k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
    for (int k = 0; k < kPartialStride; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], o);
  if ((threadIdx.x & 31) == 0)
    for (int k = 0; k < kPartialStride; ++k) s[threadIdx.x >> 5][k] = acc[k];
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot[kPartialStride];
    for (int k = 0; k < kPartialStride; ++k) tot[k] = 0.0;
    for (int wv = 0; wv < 32; ++wv)
      for (int k = 0; k < kPartialStride; ++k) tot[k] += s[wv][k];
    const float l = (float)(-tot[0]);
    *loss = accumulate ? *loss + l : l;
    if (metrics) {
      const double nk = tot[4] > 0.0 ? tot[4] : 1.0;
      metrics[0] = (float)(tot[1] / nk);
      metrics[1] = (float)(tot[2] / nk);
      metrics[2] = (float)(tot[3] / nk);
      metrics[3] = (float)tot[4];
    }
  }
}

}  // namespace

static size_t max_tiles_of(int64_t T, int32_t R, int tile_rows) {
  return (size_t)(T / tile_rows) + (size_t)R + 2;
}

size_t aero_tiles_bytes(int64_t T, int32_t R, int tile_rows) {
  return 2 * aero_align_up(max_tiles_of(T, R, tile_rows) * sizeof(int32_t), 256) + 256;
}

aero_tiles aero_carve_tiles(void* ws, int64_t T, int32_t R, int tile_rows) {
  aero_tiles t;
  const size_t mt = max_tiles_of(T, R, tile_rows);
  char* p = static_cast<char*>(ws);
  t.n_tiles = reinterpret_cast<int32_t*>(p);       p += 256;
  t.tile_row = reinterpret_cast<int32_t*>(p);      p += aero_align_up(mt * sizeof(int32_t), 256);
  t.tile_valid = reinterpret_cast<int32_t*>(p);
  t.max_tiles = (int32_t)mt;
  return t;
}

int aero_build_dense_tiles(aero_ctx* ctx, int64_t T, int tile_rows, aero_tiles tiles) {
  if (T == 0) {
    AERO_CUDA_TRY(cudaMemsetAsync(tiles.n_tiles, 0, sizeof(int32_t), ctx->stream));
    return AERO_OK;
  }
  const long long n = (T + tile_rows - 1) / tile_rows;
  const int blocks = (int)((n + 255) / 256 < 1024 ? (n + 255) / 256 : 1024);
  dense_tiles_kernel<<<blocks, 256, 0, ctx->stream>>>(T, tile_rows, tiles.tile_row, tiles.tile_valid, tiles.n_tiles,
                                                       tiles.max_tiles);
  ctx->launches += 1;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}

int aero_build_tiles(aero_ctx* ctx, int64_t T, int32_t R, const int64_t* cs, const uint8_t* keep,
                     int tile_rows, aero_tiles tiles) {
  if (R == 0 || T == 0) {
    AERO_CUDA_TRY(cudaMemsetAsync(tiles.n_tiles, 0, sizeof(int32_t), ctx->stream));
    return AERO_OK;
  }
  build_tiles_kernel<<<1, 1024, 0, ctx->stream>>>(T, R, cs, keep, tile_rows, tiles.tile_row,
                                                  tiles.tile_valid, tiles.n_tiles, tiles.max_tiles);
  ctx->launches += 1;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}

int aero_loss_finalize(aero_ctx* ctx, const double* partials, int n_partials, int stride,
                       float* loss, float* metrics, int accumulate) {
  finalize_kernel<<<1, 1024, 0, ctx->stream>>>(partials, n_partials, stride, loss, metrics, accumulate);
  ctx->launches += 1;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}
