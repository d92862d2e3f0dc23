// Decoder glue around the pyramid path for whole-model workloads (not from the paper: the public
// Llama block that the workloads name - token embedding, RMSNorm, linear layers, rotary embedding at a
// token's ORIGINAL position (Appendix A.2, "gather": a kept key keeps its position), SwiGLU, greedy
// argmax). CUDA-core kernels in fp32 arithmetic for fp32 and bf16 storage; the linear layer is a plain
// shared-memory tiled GEMM, meant for the small fp32 model whose 1e-4 tolerance rules TF32 out.
#include <cuda_bf16.h>

#include "pyr_internal.h"

namespace pyr {
namespace {

template <typename T> __device__ __forceinline__ float ld(const T* p);
template <> __device__ __forceinline__ float ld<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st(T* p, float v);
template <> __device__ __forceinline__ void st<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T>
__global__ void embed_kernel(const int32_t* ids, const T* table, T* out, int64_t tokens, int d, int vocab, int* status) {
  const int64_t t = blockIdx.x;
  int id = ids[t];
  if (id < 0 || id >= vocab) {                  // recorded, and the row is zeroed rather than read out of bounds
    if (threadIdx.x == 0 && status) atomicCAS(status, 0, (int)PYR_ERR_INVALID);
    for (int i = threadIdx.x; i < d; i += blockDim.x) st(out + t * d + i, 0.f);
    return;
  }
  for (int i = threadIdx.x; i < d; i += blockDim.x) out[t * d + i] = table[(int64_t)id * d + i];
}

// out = x / sqrt(mean(x^2) + eps) * gain, one CTA per row, the squares summed in a fixed order.
// With a row map, output row (b, i) reads x row (b, rows[b][i]): the kept rows are normalised
// straight out of the uncompacted tensor.
template <typename T>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const T* x, const T* gain, T* out, int d, float eps, RowMap map) {
  __shared__ float red[8];
  const int64_t t = blockIdx.x;
  x += (map.source_row(t) - t) * d;
  float s = 0.f;
  for (int i = threadIdx.x; i < d; i += 256) { const float v = ld(x + t * d + i); s = fmaf(v, v, s); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float r = rsqrtf(tot / (float)d + eps);
  for (int i = threadIdx.x; i < d; i += 256) st(out + t * d + i, ld(x + t * d + i) * r * ld(gain + i));
}

// y[t, n] = sum_k x[t, k] w[n, k] (+ res[t, n]); 64 x 64 output tile per CTA, 16 k per step, 4 x 4 outputs per thread
template <typename T>
__global__ void __launch_bounds__(256) linear_kernel(const T* x, const T* w, const T* res, T* y, int64_t M, int N, int K,
                                                     RowMap map) {
  __shared__ float xs[16][64 + 1], ws[16][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t m0 = (int64_t)blockIdx.y * 64;
  const int n0 = blockIdx.x * 64;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      const int r = e >> 4, kk = e & 15;
      xs[kk][r] = (m0 + r < M && k0 + kk < K) ? ld(x + (m0 + r) * K + k0 + kk) : 0.f;
      ws[kk][r] = (n0 + r < N && k0 + kk < K) ? ld(w + (int64_t)(n0 + r) * K + k0 + kk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = xs[kk][ty * 4 + i]; b[i] = ws[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t m = m0 + ty * 4 + i;
      const int n = n0 + tx * 4 + j;
      if (m < M && n < N) st(y + m * N + n, acc[i][j] + (res ? ld(res + map.source_row(m) * N + n) : 0.f));
    }
}

// rotate the pairs (i, i + D/2) of every head of token t by pos[t] * 10000^(-2i/D). One CTA per token:
// the D/2 angles are the same for all heads, so they are taken once (in double: positions reach the
// thousands and the fp32 model is held to 1e-4) and kept in shared memory as fp32 cosines and sines.
constexpr int kRopeMaxHalf = 128;
template <typename T>
__global__ void __launch_bounds__(256) rope_kernel(T* x, const int32_t* pos, int64_t tokens, int H, int D) {
  __shared__ float2 cs[kRopeMaxHalf];
  const int half = D / 2;
  const int64_t t = blockIdx.x;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    const double ang = (double)pos[t] * exp2(-2.0 * (double)i / (double)D * 13.287712379549449);   // log2(10000)
    double sn, c;
    sincos(ang, &sn, &c);
    cs[i] = make_float2((float)c, (float)sn);
  }
  __syncthreads();
  T* row = x + t * (int64_t)H * D;
  for (int e = threadIdx.x; e < H * half; e += blockDim.x) {
    const int i = e % half, h = e / half;
    T* p = row + h * D;
    const float a = ld(p + i), b = ld(p + i + half);
    const float2 w = cs[i];
    st(p + i, a * w.x - b * w.y);
    st(p + i + half, b * w.x + a * w.y);
  }
}

template <typename T>
__global__ void swiglu_kernel(const T* g, const T* u, T* out, int64_t n) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n) return;
  const float gv = ld(g + e);
  st(out + e, gv / (1.f + expf(-gv)) * ld(u + e));
}

// argmax of every row, the lowest index winning ties; one CTA per row
template <typename T>
__global__ void __launch_bounds__(256) argmax_kernel(const T* x, int32_t* out, int n) {
  __shared__ float bv[256];
  __shared__ int bi[256];
  const int64_t r = blockIdx.x;
  float best = -INFINITY;
  int idx = 0x7fffffff;
  for (int i = threadIdx.x; i < n; i += 256) {
    const float v = ld(x + r * n + i);
    if (v > best || (v == best && i < idx)) { best = v; idx = i; }
  }
  bv[threadIdx.x] = best; bi[threadIdx.x] = idx;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (threadIdx.x < s) {
      const float v = bv[threadIdx.x + s];
      const int i = bi[threadIdx.x + s];
      if (v > bv[threadIdx.x] || (v == bv[threadIdx.x] && i < bi[threadIdx.x])) { bv[threadIdx.x] = v; bi[threadIdx.x] = i; }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) out[r] = bi[0];
}

template <typename F32, typename BF16>
cudaError_t by_dtype(int dtype, F32 f32, BF16 bf16) {
  if (dtype == PYR_F32) f32(); else if (dtype == PYR_BF16) bf16(); else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_glue_embed(const int32_t* ids, const void* table, void* out, int64_t tokens, int d, int vocab,
                              int dtype, int* status, cudaStream_t s) {
  if (tokens == 0) return cudaSuccess;
  return by_dtype(dtype,
      [&] { embed_kernel<float><<<(unsigned)tokens, 128, 0, s>>>(ids, (const float*)table, (float*)out, tokens, d, vocab, status); },
      [&] { embed_kernel<__nv_bfloat16><<<(unsigned)tokens, 128, 0, s>>>(ids, (const __nv_bfloat16*)table, (__nv_bfloat16*)out, tokens, d, vocab, status); });
}
cudaError_t launch_glue_rmsnorm(const void* x, const void* gain, void* out, int64_t tokens, int d, float eps, int dtype,
                                const RowMap& map, cudaStream_t s) {
  if (tokens == 0) return cudaSuccess;
  return by_dtype(dtype,
      [&] { rmsnorm_kernel<float><<<(unsigned)tokens, 256, 0, s>>>((const float*)x, (const float*)gain, (float*)out, d, eps, map); },
      [&] { rmsnorm_kernel<__nv_bfloat16><<<(unsigned)tokens, 256, 0, s>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)gain, (__nv_bfloat16*)out, d, eps, map); });
}
cudaError_t launch_glue_linear(const void* x, const void* w, const void* res, void* y, int64_t M, int N, int K, int dtype,
                               const RowMap& map, cudaStream_t s) {
  if (M == 0 || N == 0) return cudaSuccess;
  dim3 grid((N + 63) / 64, (unsigned)((M + 63) / 64));
  return by_dtype(dtype,
      [&] { linear_kernel<float><<<grid, 256, 0, s>>>((const float*)x, (const float*)w, (const float*)res, (float*)y, M, N, K, map); },
      [&] { linear_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w, (const __nv_bfloat16*)res, (__nv_bfloat16*)y, M, N, K, map); });
}
cudaError_t launch_glue_rope(void* x, const int32_t* pos, int64_t tokens, int H, int D, int dtype, cudaStream_t s) {
  if (tokens == 0) return cudaSuccess;
  if (D / 2 > kRopeMaxHalf || tokens > 0x7fffffffLL) return cudaErrorInvalidValue;
  const unsigned blocks = (unsigned)tokens;
  return by_dtype(dtype,
      [&] { rope_kernel<float><<<blocks, 256, 0, s>>>((float*)x, pos, tokens, H, D); },
      [&] { rope_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>((__nv_bfloat16*)x, pos, tokens, H, D); });
}
cudaError_t launch_glue_swiglu(const void* g, const void* u, void* out, int64_t n, int dtype, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  const unsigned blocks = (unsigned)((n + 255) / 256);
  return by_dtype(dtype,
      [&] { swiglu_kernel<float><<<blocks, 256, 0, s>>>((const float*)g, (const float*)u, (float*)out, n); },
      [&] { swiglu_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>((const __nv_bfloat16*)g, (const __nv_bfloat16*)u, (__nv_bfloat16*)out, n); });
}
cudaError_t launch_glue_argmax(const void* x, int32_t* out, int64_t rows, int n, int dtype, cudaStream_t s) {
  if (rows == 0) return cudaSuccess;
  return by_dtype(dtype,
      [&] { argmax_kernel<float><<<(unsigned)rows, 256, 0, s>>>((const float*)x, out, n); },
      [&] { argmax_kernel<__nv_bfloat16><<<(unsigned)rows, 256, 0, s>>>((const __nv_bfloat16*)x, out, n); });
}

}  // namespace pyr
