// Generation-phase update of a layer's PvC (Algorithm 1 with
// KV = cat([PvC_past, KV]); Section 4.1, Generation Phase): the ensemble score
// of the cache's context rows from the attention weights of the sliding recent
// window, taken over the cache as it is now. Window query i (oldest first) sees
// the context and the window rows up to its own.
//
// bf16 with head dim 128 runs on the warp-level tensor-core MMAs (gen_score_mma_kernel below);
// the CUDA-core kernel serves every other dtype and head dim: a thread owns one window
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

// ------------------------------------------------------------------ bf16, head dim 128: warp-level MMAs
// A CTA takes 128 window queries of one (sequence, head): 8 warps x 16 rows, each warp's rows the A
// operand of m16n8k16 MMAs held in registers for the whole kernel. The cache rows of the KV head
// stream through shared memory in tiles of 64 (cp.async, two buffers, rows padded to 272 bytes so
// that ldmatrix meets no bank conflict). Two passes over the cache as in the kernel above: the rows'
// log-sum-exp on the accumulator fragments first, then w_i 2^(s - lse_i) summed down the columns -
// within a thread (its two rows), across the warp's eight row groups by a fixed shuffle tree, across
// the eight warps in order - so the scores are bit-reproducible.
constexpr int kMq = 128, kMk = 64, kMkStride = 272;

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

__global__ void __launch_bounds__(256) gen_score_mma_kernel(GenScoreArgs a) {
  constexpr int D = 128;
  __shared__ __align__(16) uint8_t ktile[2][kMk * kMkStride];
  __shared__ float wsum[8][kMk];
  const int bh = blockIdx.x, qt = blockIdx.y;
  const int b = bh / a.Hq, h = bh % a.Hq;
  const int g = h / (a.Hq / a.Hkv);
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int gq = lane >> 2, tq = lane & 3;
  const int c = a.c;
  const __nv_bfloat16* kbase = static_cast<const __nv_bfloat16*>(a.kc) + ((int64_t)b * a.Hkv + g) * (int64_t)a.cap * D;
  const float sc2 = a.scale * kLog2e;

  // window rows of this thread: i0 and i0 + 8; A fragments of both for the 8 k-steps
  const int i0 = qt * kMq + warp * 16 + gq, i1 = i0 + 8;
  uint32_t qa[8][4];
  {
    const __nv_bfloat16* qw = static_cast<const __nv_bfloat16*>(a.qwin);
    auto qrow = [&](int i) {
      const int slot = (a.start + i) % a.R;
      return reinterpret_cast<const uint32_t*>(qw + (((int64_t)b * a.R + slot) * a.Hq + h) * (int64_t)D);
    };
    const uint32_t* r0 = qrow(i0 < a.Lw ? i0 : 0);
    const uint32_t* r1 = qrow(i1 < a.Lw ? i1 : 0);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = i0 < a.Lw ? r0[ks * 8 + tq] : 0u;          // d = 16 ks + 2 tq, + 1
      qa[ks][1] = i1 < a.Lw ? r1[ks * 8 + tq] : 0u;
      qa[ks][2] = i0 < a.Lw ? r0[ks * 8 + 4 + tq] : 0u;      // d = 16 ks + 8 + 2 tq, + 1
      qa[ks][3] = i1 < a.Lw ? r1[ks * 8 + 4 + tq] : 0u;
    }
  }
  const float w0 = i0 < a.Lw ? a.w[i0] : 0.f, w1 = i1 < a.Lw ? a.w[i1] : 0.f;
  const int last0 = c + i0, last1 = c + i1;           // the newest cache row each query sees

  // ldmatrix: lane supplies row (lane & 7) of matrix (lane >> 3): matrices (keys 0-7, d lo), (keys 0-7, d hi),
  // (keys 8-15, d lo), (keys 8-15, d hi) of a 16-key, 16-d block
  const uint32_t lm_off = (uint32_t)(((lane >> 4) * 8 + (lane & 7)) * kMkStride + ((lane >> 3) & 1) * 16);

  auto issue_tile = [&](int j0, int buf) {
    for (int e = t; e < kMk * 16; e += 256) {
      const int row = e >> 4, ch = e & 15;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&ktile[buf][row * kMkStride + ch * 16]);
      if (j0 + row < a.len) cp_async16(dst, kbase + (int64_t)(j0 + row) * D + ch * 8);
      else *reinterpret_cast<uint4*>(&ktile[buf][row * kMkStride + ch * 16]) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // S of this warp's 16 rows x the tile's 64 keys: sc[nb][0,1] = row i0, keys 8 nb + 2 tq (+1); [2,3] = row i1
  auto tile_scores = [&](int buf, float (*sc)[4]) {
    const uint32_t kb = (uint32_t)__cvta_generic_to_shared(&ktile[buf][0]) + lm_off;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
#pragma unroll
    for (int np = 0; np < 4; ++np) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t bf[4];
        ldsm4(kb + np * 16 * kMkStride + ks * 32, bf);
        mma16816(sc[2 * np], qa[ks], bf[0], bf[1]);
        mma16816(sc[2 * np + 1], qa[ks], bf[2], bf[3]);
      }
    }
  };

  // pass 1: log2-domain log-sum-exp of rows i0 and i1 over the cache rows they see
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const int ntiles = (a.len + kMk - 1) / kMk;
  issue_tile(0, 0);
  for (int tI = 0; tI < ntiles; ++tI) {
    if (tI + 1 < ntiles) issue_tile((tI + 1) * kMk, (tI + 1) & 1);
    if (tI + 1 < ntiles) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    float sc[8][4];
    tile_scores(tI & 1, sc);
    const int j0 = tI * kMk;
    float x0 = -INFINITY, x1 = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int j = j0 + nb * 8 + tq * 2 + e;
        sc[nb][e] = (j <= last0 && j < a.len) ? sc[nb][e] * sc2 : -INFINITY;
        sc[nb][2 + e] = (j <= last1 && j < a.len) ? sc[nb][2 + e] * sc2 : -INFINITY;
        x0 = fmaxf(x0, sc[nb][e]);
        x1 = fmaxf(x1, sc[nb][2 + e]);
      }
    }
    x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 1)); x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 2));
    x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 1)); x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 2));
    const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);
    float s0 = 0.f, s1 = 0.f;
    if (n0 > -INFINITY) {
#pragma unroll
      for (int nb = 0; nb < 8; ++nb) s0 += exp2f(sc[nb][0] - n0) + exp2f(sc[nb][1] - n0);
      l0 = l0 * exp2f(m0 - n0) + s0;
      m0 = n0;
    }
    if (n1 > -INFINITY) {
#pragma unroll
      for (int nb = 0; nb < 8; ++nb) s1 += exp2f(sc[nb][2] - n1) + exp2f(sc[nb][3] - n1);
      l1 = l1 * exp2f(m1 - n1) + s1;
      m1 = n1;
    }
    __syncthreads();      // the buffer this tile used is refilled two tiles on
  }
  // the row sums are spread over the four threads of a row
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float lse0 = m0 + log2f(l0), lse1 = m1 + log2f(l1);

  // pass 2: E[j] = sum_i w_i 2^(s_ij - lse_i) over the CTA's 128 queries, context rows only
  float* part = a.part + (((int64_t)b * a.Hq + h) * gridDim.y + qt) * (int64_t)c;
  const int ctiles = (c + kMk - 1) / kMk;
  issue_tile(0, 0);
  for (int tI = 0; tI < ctiles; ++tI) {
    if (tI + 1 < ctiles) issue_tile((tI + 1) * kMk, (tI + 1) & 1);
    if (tI + 1 < ctiles) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    float sc[8][4];
    tile_scores(tI & 1, sc);
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        // every context row is visible to every window query
        float v = w0 * exp2f(sc[nb][e] * sc2 - lse0) + w1 * exp2f(sc[nb][2 + e] * sc2 - lse1);
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (gq == 0) wsum[warp][nb * 8 + tq * 2 + e] = v;
      }
    }
    __syncthreads();
    const int j0 = tI * kMk;
    if (t < kMk && j0 + t < c) {
      float v = 0.f;
#pragma unroll
      for (int wI = 0; wI < 8; ++wI) v += wsum[wI][t];
      part[j0 + t] = v;
    }
    // (the next iteration's first barrier separates these reads of wsum from its writes)
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

// query tiles of the finer-grained of the two kernels: what the per-head partial buffer is sized for
int gen_score_qtiles(int Lw) { return (Lw + kMq - 1) / kMq; }

cudaError_t launch_gen_score(const GenScoreArgs& a, cudaStream_t s) {
  if (a.c <= 0 || a.Lw <= 0) return cudaSuccess;
  const bool mma = a.dtype == PYR_BF16 && a.D == 128;
  const int qtiles = mma ? (a.Lw + kMq - 1) / kMq : (a.Lw + kGenThreads - 1) / kGenThreads;
  dim3 grid(a.B * a.Hq, qtiles);
  if (mma) gen_score_mma_kernel<<<grid, 256, 0, s>>>(a);
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
