// CUDA-core (fp32 FMA) causal attention and recent-window score.
//
// This is the path for fp32 inputs, whose 1e-4 output tolerance is tighter
// than a TF32 tensor-core product allows, and the on-device cross-check of the
// tcgen05 path for bf16. Algorithm 1: "compute attention weights of KV" and
// "A_e <- weighted_avg(A[-L:, :-L], dim=-2)".
#include <cuda_bf16.h>

#include "pyr_internal.h"

namespace pyr {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <class T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}
template <class T> __device__ __forceinline__ void stf(T* p, float x);
template <> __device__ __forceinline__ void stf<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float x) {
  *p = __float2bfloat16_rn(x);
}

constexpr int BM = 32;   // query rows per CTA
constexpr int BN = 32;   // keys per tile

// 128 threads: thread t owns query row r = t / 4 of the tile; the 4 threads of
// a row split the 32 keys of a tile (8 each) and the D output columns
// (interleaved by 4).
template <class T, int D>
__global__ void __launch_bounds__(128) prefill_simt_kernel(PrefillArgs a) {
  extern __shared__ float smem_f[];
  float (*Qs)[D + 1] = reinterpret_cast<float (*)[D + 1]>(smem_f);
  float (*Ks)[D + 1] = reinterpret_cast<float (*)[D + 1]>(smem_f + BM * (D + 1));
  float (*Vs)[D] = reinterpret_cast<float (*)[D]>(smem_f + (BM + BN) * (D + 1));
  float (*Ps)[BN + 1] = reinterpret_cast<float (*)[BN + 1]>(smem_f + (BM + BN) * (D + 1) + BN * D);

  const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int g = h / (a.Hq / a.Hkv);
  const int t = threadIdx.x, r = t >> 2, part = t & 3;
  const int row0 = tile * BM;
  const int n = a.n;
  const T* q = static_cast<const T*>(a.q) + b * a.qsb + h * a.qsh;
  const T* k = static_cast<const T*>(a.k) + b * a.ksb + g * a.ksh;
  const T* v = static_cast<const T*>(a.v) + b * a.ksb + g * a.ksh;
  const float sc2 = a.scale * kLog2e;

  for (int e = t; e < BM * D; e += 128) {
    int rr = e / D, d = e % D;
    Qs[rr][d] = (row0 + rr < n) ? ldf(q + (int64_t)(row0 + rr) * a.qsn + d) * sc2 : 0.f;
  }

  constexpr int DC = D / 4;
  float acc[DC];
#pragma unroll
  for (int i = 0; i < DC; ++i) acc[i] = 0.f;
  float m = -INFINITY, l = 0.f;
  const int i_glob = row0 + r;
  const int last_key = min(row0 + BM, n);   // keys [0, last_key) can be visible to this tile

  for (int k0 = 0; k0 < last_key; k0 += BN) {
    __syncthreads();
    for (int e = t; e < BN * D; e += 128) {
      int rr = e / D, d = e % D;
      bool ok = k0 + rr < n;
      Ks[rr][d] = ok ? ldf(k + (int64_t)(k0 + rr) * a.ksn + d) : 0.f;
      Vs[rr][d] = ok ? ldf(v + (int64_t)(k0 + rr) * a.ksn + d) : 0.f;
    }
    __syncthreads();
    float s[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) s[jj] = 0.f;
    for (int d = 0; d < D; ++d) {
      float qv = Qs[r][d];
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) s[jj] = fmaf(qv, Ks[part * 8 + jj][d], s[jj]);
    }
    float mx = -INFINITY;
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) {
      int j = k0 + part * 8 + jj;
      if (j > i_glob || j >= n) s[jj] = -INFINITY;
      mx = fmaxf(mx, s[jj]);
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m, mx);
    // every row sees key 0 in the first tile, so m_new is finite from then on
    const float corr = exp2f(m - m_new);
    float ps = 0.f;
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) {
      float p = exp2f(s[jj] - m_new);
      Ps[r][part * 8 + jj] = p;
      ps += p;
    }
    ps += __shfl_xor_sync(0xffffffffu, ps, 1);
    ps += __shfl_xor_sync(0xffffffffu, ps, 2);
    l = l * corr + ps;
    m = m_new;
    __syncwarp();   // a row's 4 threads sit in one warp; Ps[r][*] is theirs alone
#pragma unroll
    for (int i = 0; i < DC; ++i) acc[i] *= corr;
    for (int j = 0; j < BN; ++j) {
      float p = Ps[r][j];
#pragma unroll
      for (int i = 0; i < DC; ++i) acc[i] = fmaf(p, Vs[j][i * 4 + part], acc[i]);
    }
  }
  if (i_glob < n) {
    const float inv = 1.f / l;
    T* o = static_cast<T*>(a.out) + b * a.osb + h * a.osh + (int64_t)i_glob * a.osn;
#pragma unroll
    for (int i = 0; i < DC; ++i) stf(o + i * 4 + part, acc[i] * inv);
    if (part == 0) a.lse[((int64_t)b * a.Hq + h) * n + i_glob] = (m + log2f(l)) * kLn2;
  }
}

// score[b,g,j] = (1/heads) sum_{h in g} sum_i w_i exp(scale q_{c+i}.k_j - lse_{c+i}).
// 128 threads: thread t owns key j = tile*32 + t/4 and the recent queries
// i = t%4 (mod 4). Sums run in a fixed order: heads ascending, queries
// ascending, then a fixed shuffle tree over the 4 partial sums.
template <class T, int D>
__global__ void __launch_bounds__(128) score_simt_kernel(PrefillArgs a) {
  __shared__ float Qs[32][D + 1];
  __shared__ float Ks[32][D + 1];
  __shared__ float bias[32];

  const int tile = blockIdx.x, gsel = blockIdx.y, b = blockIdx.z;
  const int t = threadIdx.x, jl = t >> 2, part = t & 3;
  const int n = a.n, L = a.L, c = n - L;
  const int heads = a.Hq / a.G;
  const int rep = a.Hq / a.Hkv;
  const float sc2 = a.scale * kLog2e;
  const int j0 = tile * 32;
  float acc = 0.f;
  int g_loaded = -1;
  for (int hh = 0; hh < heads; ++hh) {
    const int h = gsel * heads + hh;
    const int g = h / rep;
    const T* q = static_cast<const T*>(a.q) + b * a.qsb + h * a.qsh;
    const T* k = static_cast<const T*>(a.k) + b * a.ksb + g * a.ksh;
    const float* lse = a.lse + ((int64_t)b * a.Hq + h) * n;
    if (g != g_loaded) {
      __syncthreads();
      for (int e = t; e < 32 * D; e += 128) {
        int rr = e / D, d = e % D;
        Ks[rr][d] = (j0 + rr < c) ? ldf(k + (int64_t)(j0 + rr) * a.ksn + d) : 0.f;
      }
      g_loaded = g;
    }
    for (int i0 = 0; i0 < L; i0 += 32) {
      __syncthreads();
      for (int e = t; e < 32 * D; e += 128) {
        int rr = e / D, d = e % D;
        Qs[rr][d] = (i0 + rr < L) ? ldf(q + (int64_t)(c + i0 + rr) * a.qsn + d) * sc2 : 0.f;
      }
      if (t < 32) bias[t] = (i0 + t < L) ? log2f(a.w[i0 + t]) - lse[c + i0 + t] * kLog2e : -INFINITY;
      __syncthreads();
      for (int ii = part; ii < 32; ii += 4) {
        float s = 0.f;
        for (int d = 0; d < D; ++d) s = fmaf(Qs[ii][d], Ks[jl][d], s);
        acc += exp2f(s + bias[ii]);
      }
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  acc += __shfl_xor_sync(0xffffffffu, acc, 2);
  if (part == 0 && j0 + jl < c)
    a.score[((int64_t)b * a.G + gsel) * c + j0 + jl] = acc * (1.f / (float)heads);
}

template <class T, int D>
cudaError_t run_prefill_simt(const PrefillArgs& a, cudaStream_t s) {
  constexpr size_t smem = sizeof(float) * ((BM + BN) * (D + 1) + BN * D + BM * (BN + 1));
  cudaError_t e = cudaFuncSetAttribute(prefill_simt_kernel<T, D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((a.n + BM - 1) / BM, a.Hq, a.B);
  prefill_simt_kernel<T, D><<<grid, 128, smem, s>>>(a);
  return cudaGetLastError();
}

template <class T, int D>
cudaError_t run_score_simt(const PrefillArgs& a, cudaStream_t s) {
  const int c = a.n - a.L;
  dim3 grid((c + 31) / 32, a.G, a.B);
  score_simt_kernel<T, D><<<grid, 128, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill_simt(const PrefillArgs& a, cudaStream_t s) {
  if (a.dtype == PYR_F32)
    return a.D == 64 ? run_prefill_simt<float, 64>(a, s) : run_prefill_simt<float, 128>(a, s);
  return a.D == 64 ? run_prefill_simt<__nv_bfloat16, 64>(a, s)
                   : run_prefill_simt<__nv_bfloat16, 128>(a, s);
}

cudaError_t launch_score_simt(const PrefillArgs& a, cudaStream_t s) {
  if (a.n - a.L <= 0) return cudaSuccess;
  if (a.dtype == PYR_F32)
    return a.D == 64 ? run_score_simt<float, 64>(a, s) : run_score_simt<float, 128>(a, s);
  return a.D == 64 ? run_score_simt<__nv_bfloat16, 64>(a, s) : run_score_simt<__nv_bfloat16, 128>(a, s);
}

}  // namespace pyr
