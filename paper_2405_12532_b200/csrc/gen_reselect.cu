// Generation-phase update of a layer's PvC (Algorithm 1 with
// KV = cat([PvC_past, KV]); Section 4.1, Generation Phase): the ensemble score
// of the cache's context rows from the attention weights of the sliding recent
// window, taken over the cache as it is now. Window query i (oldest first) sees
// the context and the window rows up to its own.
//
// CUDA-core kernels for every dtype and head dim: a thread owns one window
// query, keeps it in registers and walks the cache twice - once for the row's
// log-sum-exp, once for the weighted column sums, which are reduced over the
// block's 256 queries in a fixed order (warp tree, then warps in order): the
// scores are bit-reproducible. The top-k and the in-place row compaction that
// follow are the prefill step's kernels.
#include <cuda_bf16.h>

#include "pyr_internal.h"

namespace pyr {
namespace {

constexpr int kGenThreads = 256;   // window queries per CTA
constexpr int kGenKeys = 32;       // cache rows per shared-memory tile
constexpr float kLog2e = 1.4426950408889634f;

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T, int D>
__global__ void __launch_bounds__(kGenThreads) gen_score_kernel(GenScoreArgs a) {
  __shared__ float ktile[kGenKeys][D];
  __shared__ float wsum[kGenThreads / 32][kGenKeys];
  const int bh = blockIdx.x, qt = blockIdx.y;
  const int b = bh / a.Hq, h = bh % a.Hq;
  const int g = h / (a.Hq / a.Hkv);
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int i = qt * kGenThreads + t;                 // window query of this thread
  const bool live = i < a.Lw;
  const int c = a.c;
  const T* kbase = static_cast<const T*>(a.kc) + ((int64_t)b * a.Hkv + g) * (int64_t)a.cap * D;

  float q[D];
  {
    const int slot = (a.start + (live ? i : 0)) % a.R;
    const T* qp = static_cast<const T*>(a.qwin) + (((int64_t)b * a.R + slot) * a.Hq + h) * (int64_t)D;
    const float sc = a.scale * kLog2e;
#pragma unroll
    for (int d = 0; d < D; ++d) q[d] = to_f32(qp[d]) * sc;
  }
  const int last = c + i;                             // the newest cache row this query sees
  const float wi = live ? a.w[i] : 0.f;

  auto load_tile = [&](int j0) {
    __syncthreads();
    for (int e = t; e < kGenKeys * D; e += kGenThreads) {
      const int kk = e / D, d = e % D;
      const int j = j0 + kk;
      ktile[kk][d] = j < a.len ? to_f32(kbase[(int64_t)j * D + d]) : 0.f;
    }
    __syncthreads();
  };

  // pass 1: log2-domain log-sum-exp of the row over the cache rows it sees
  float m = -INFINITY, l = 0.f;
  for (int j0 = 0; j0 < a.len; j0 += kGenKeys) {
    load_tile(j0);
    float s[kGenKeys];
    float tm = -INFINITY;
#pragma unroll
    for (int kk = 0; kk < kGenKeys; ++kk) {
      float acc = 0.f;
#pragma unroll
      for (int d = 0; d < D; ++d) acc = fmaf(q[d], ktile[kk][d], acc);
      s[kk] = (j0 + kk <= last && j0 + kk < a.len) ? acc : -INFINITY;
      tm = fmaxf(tm, s[kk]);
    }
    if (tm > -INFINITY) {
      const float mn = fmaxf(m, tm);
      float add = 0.f;
#pragma unroll
      for (int kk = 0; kk < kGenKeys; ++kk) add += exp2f(s[kk] - mn);
      l = l * exp2f(m - mn) + add;
      m = mn;
    }
  }
  const float lse2 = m + log2f(l);

  // pass 2: E[j] = sum_i w_i 2^(s_ij - lse_i) over the block's queries, context rows only
  float* part = a.part + (((int64_t)b * a.Hq + h) * gridDim.y + qt) * (int64_t)c;
  for (int j0 = 0; j0 < c; j0 += kGenKeys) {
    load_tile(j0);
#pragma unroll
    for (int kk = 0; kk < kGenKeys; ++kk) {
      float acc = 0.f;
#pragma unroll
      for (int d = 0; d < D; ++d) acc = fmaf(q[d], ktile[kk][d], acc);
      float v = live ? wi * exp2f(acc - lse2) : 0.f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) wsum[warp][kk] = v;
    }
    __syncthreads();
    if (t < kGenKeys && j0 + t < c) {
      float v = 0.f;
#pragma unroll
      for (int wI = 0; wI < kGenThreads / 32; ++wI) v += wsum[wI][t];
      part[j0 + t] = v;
    }
  }
}

// score[b, g, j] = mean over the query heads of group g of the sum over the
// window's query tiles of the per-head partial scores, in a fixed order.
__global__ void __launch_bounds__(256) gen_pool_kernel(GenScoreArgs a, int qtiles) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t total = (int64_t)a.B * a.G * a.c;
  if (e >= total) return;
  const int j = (int)(e % a.c);
  const int g = (int)((e / a.c) % a.G);
  const int b = (int)(e / ((int64_t)a.c * a.G));
  const int per = a.Hq / a.G;
  float v = 0.f;
  for (int hh = 0; hh < per; ++hh) {
    const int h = g * per + hh;
    for (int qt = 0; qt < qtiles; ++qt) v += a.part[(((int64_t)b * a.Hq + h) * qtiles + qt) * (int64_t)a.c + j];
  }
  a.score[e] = v / (float)per;
}

// Rows [r0, r0 + rows) of a strided [B, rows, row_bytes] source to a strided destination, 16 bytes per thread.
__global__ void __launch_bounds__(256) copy_rows_kernel(const char* src, char* dst, int64_t src_sb, int64_t src_sn,
                                                        int64_t dst_sb, int64_t dst_sn, int B, int rows, int lanes) {
  const int64_t total = (int64_t)B * rows * lanes;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int lane = (int)(e % lanes);
    const int r = (int)((e / lanes) % rows);
    const int b = (int)(e / ((int64_t)lanes * rows));
    *reinterpret_cast<uint4*>(dst + b * dst_sb + r * dst_sn + (int64_t)lane * 16) =
        *reinterpret_cast<const uint4*>(src + b * src_sb + r * src_sn + (int64_t)lane * 16);
  }
}

}  // namespace

int gen_score_qtiles(int Lw) { return (Lw + kGenThreads - 1) / kGenThreads; }

cudaError_t launch_gen_score(const GenScoreArgs& a, cudaStream_t s) {
  if (a.c <= 0 || a.Lw <= 0) return cudaSuccess;
  const int qtiles = gen_score_qtiles(a.Lw);
  dim3 grid(a.B * a.Hq, qtiles);
  if (a.dtype == PYR_BF16 && a.D == 128) gen_score_kernel<__nv_bfloat16, 128><<<grid, kGenThreads, 0, s>>>(a);
  else if (a.dtype == PYR_BF16 && a.D == 64) gen_score_kernel<__nv_bfloat16, 64><<<grid, kGenThreads, 0, s>>>(a);
  else if (a.dtype == PYR_F32 && a.D == 128) gen_score_kernel<float, 128><<<grid, kGenThreads, 0, s>>>(a);
  else if (a.dtype == PYR_F32 && a.D == 64) gen_score_kernel<float, 64><<<grid, kGenThreads, 0, s>>>(a);
  else return cudaErrorInvalidValue;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int64_t total = (int64_t)a.B * a.G * a.c;
  gen_pool_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(a, qtiles);
  return cudaGetLastError();
}

cudaError_t launch_copy_rows(const void* src, void* dst, int64_t src_sb, int64_t src_sn, int64_t dst_sb,
                             int64_t dst_sn, int B, int rows, int row_bytes, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  const int lanes = row_bytes / 16;
  const int64_t total = (int64_t)B * rows * lanes;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 4096) blocks = 4096;
  copy_rows_kernel<<<(unsigned)blocks, 256, 0, s>>>(static_cast<const char*>(src), static_cast<char*>(dst), src_sb,
                                                    src_sn, dst_sb, dst_sn, B, rows, lanes);
  return cudaGetLastError();
}

}  // namespace pyr
