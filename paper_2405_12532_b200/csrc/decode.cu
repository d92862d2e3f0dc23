// Generation-phase attention over one layer's compressed cache (Section 4.1:
// the generation phase reuses the smaller initial KV cache). One new query per
// (sequence, head) streams the layer's K and V once: the kernel is bound by
// HBM bandwidth, so rows are split across CTAs (split-K) and each lane keeps
// 16-byte loads of several rows in flight.
#include <cuda_bf16.h>

#include "pyr_internal.h"

namespace pyr {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kThreads = 256;
constexpr int kUnroll = 4;

template <class T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
  static constexpr int per16 = 8;
  static __device__ __forceinline__ void unpack(const uint4& r, float* f) {
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
    f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
    f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};
template <> struct Elem<float> {
  static constexpr int per16 = 4;
  static __device__ __forceinline__ void unpack(const uint4& r, float* f) {
    f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
    f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
  }
  static __device__ __forceinline__ void store(float* p, float x) { *p = x; }
};

// grid (splits, Hq / R, B). A CTA serves R consecutive query heads that share
// one KV head. RG = lanes per cache row (16 bytes each); the CTA's 256 threads
// form NG = 256 / RG row groups, group i taking rows start+i, start+i+NG, ...
template <class T, int D, int R>
__global__ void __launch_bounds__(kThreads) decode_kernel(DecodeArgs a) {
  constexpr int EPL = Elem<T>::per16;
  constexpr int RG = D / EPL;
  constexpr int NG = kThreads / RG;
  extern __shared__ float red[];   // [NG][R][D + 2]

  const int split = blockIdx.x, hy = blockIdx.y, b = blockIdx.z;
  const int h0 = hy * R;
  const int rep = a.Hq / a.Hkv;
  const int g = h0 / rep;
  const int t = threadIdx.x, grp = t / RG, ln = t % RG;
  // lanes of this row group: groups of one warp may leave the row loop at different times
  const unsigned gmask = RG == 32 ? 0xffffffffu : (((1u << (RG % 32)) - 1u) << ((t % 32) / RG * RG));
  const int total = a.len + 1;
  const int start = split * a.rows_per_split;
  const int end = min(start + a.rows_per_split, total);

  const size_t row_bytes = (size_t)D * sizeof(T);
  char* kc = static_cast<char*>(a.kc) + ((size_t)b * a.Hkv + g) * a.cap * row_bytes;
  char* vc = static_cast<char*>(a.vc) + ((size_t)b * a.Hkv + g) * a.cap * row_bytes;
  const char* kn = static_cast<const char*>(a.k_new) + ((size_t)b * a.Hkv + g) * row_bytes;
  const char* vn = static_cast<const char*>(a.v_new) + ((size_t)b * a.Hkv + g) * row_bytes;
  const bool appender = h0 == g * rep;   // first head group of this KV head stores the new row

  float q[R][EPL];
  const float sc2 = a.scale * kLog2e;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const uint4 raw = *reinterpret_cast<const uint4*>(static_cast<const char*>(a.q) +
                                                      ((size_t)b * a.Hq + h0 + r) * row_bytes + ln * 16);
    Elem<T>::unpack(raw, q[r]);
#pragma unroll
    for (int e = 0; e < EPL; ++e) q[r][e] *= sc2;
  }
  float m[R], l[R], acc[R][EPL];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[r][e] = 0.f;
  }

  for (int row = start + grp; row < end; row += NG * kUnroll) {
    uint4 kr[kUnroll], vr[kUnroll];
    bool ok[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int rw = row + u * NG;
      ok[u] = rw < end;
      if (ok[u]) {
        const bool fresh = rw == a.len;
        const char* ks = fresh ? kn : kc + (size_t)rw * row_bytes;
        const char* vs = fresh ? vn : vc + (size_t)rw * row_bytes;
        kr[u] = *reinterpret_cast<const uint4*>(ks + ln * 16);
        vr[u] = *reinterpret_cast<const uint4*>(vs + ln * 16);
        if (fresh && appender) {
          *reinterpret_cast<uint4*>(kc + (size_t)rw * row_bytes + ln * 16) = kr[u];
          *reinterpret_cast<uint4*>(vc + (size_t)rw * row_bytes + ln * 16) = vr[u];
        }
      } else {
        kr[u] = make_uint4(0, 0, 0, 0);
        vr[u] = make_uint4(0, 0, 0, 0);
      }
    }
    float kf[kUnroll][EPL], vf[kUnroll][EPL];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) { Elem<T>::unpack(kr[u], kf[u]); Elem<T>::unpack(vr[u], vf[u]); }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float s[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) d = fmaf(q[r][e], kf[u][e], d);
#pragma unroll
        for (int o = RG / 2; o > 0; o >>= 1) d += __shfl_xor_sync(gmask, d, o);
        s[u] = ok[u] ? d : -INFINITY;
      }
      float mx = s[0];
#pragma unroll
      for (int u = 1; u < kUnroll; ++u) mx = fmaxf(mx, s[u]);
      const float m_new = fmaxf(m[r], mx);      // finite: row `row` itself is valid
      const float corr = exp2f(m[r] - m_new);
      float p[kUnroll], ps = 0.f;
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) { p[u] = exp2f(s[u] - m_new); ps += p[u]; }
      l[r] = l[r] * corr + ps;
      m[r] = m_new;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        float x = acc[r][e] * corr;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) x = fmaf(p[u], vf[u][e], x);
        acc[r][e] = x;
      }
    }
  }

  // combine the NG row groups in a fixed order
#pragma unroll
  for (int r = 0; r < R; ++r) {
    float* dst = red + ((size_t)grp * R + r) * (D + 2);
#pragma unroll
    for (int e = 0; e < EPL; ++e) dst[ln * EPL + e] = acc[r][e];
    if (ln == 0) { dst[D] = m[r]; dst[D + 1] = l[r]; }
  }
  __syncthreads();
  for (int o = t; o < R * D; o += kThreads) {
    const int r = o / D, d = o % D;
    float M = -INFINITY;
    for (int gI = 0; gI < NG; ++gI) M = fmaxf(M, red[((size_t)gI * R + r) * (D + 2) + D]);
    float num = 0.f, den = 0.f;
    for (int gI = 0; gI < NG; ++gI) {
      const float* src = red + ((size_t)gI * R + r) * (D + 2);
      const float w = exp2f(src[D] - M);
      num = fmaf(w, src[d], num);
      den = fmaf(w, src[D + 1], den);
    }
    const int h = h0 + r;
    if (a.splits == 1) {
      Elem<T>::store(static_cast<T*>(a.out) + ((size_t)b * a.Hq + h) * D + d, num / den);
    } else {
      const size_t pi = ((size_t)b * a.Hq + h) * a.splits + split;
      a.part_acc[pi * D + d] = num;
      if (d == 0) { a.part_ml[pi * 2] = M; a.part_ml[pi * 2 + 1] = den; }
    }
  }
}

// Merge the splits of one (sequence, head) in ascending split order.
template <class T, int D>
__global__ void __launch_bounds__(D) decode_combine_kernel(DecodeArgs a) {
  const int bh = blockIdx.x, d = threadIdx.x;
  const float* ml = a.part_ml + (size_t)bh * a.splits * 2;
  const float* pa = a.part_acc + (size_t)bh * a.splits * D;
  float M = -INFINITY;
  for (int s = 0; s < a.splits; ++s) M = fmaxf(M, ml[s * 2]);
  float num = 0.f, den = 0.f;
  for (int s = 0; s < a.splits; ++s) {
    const float w = exp2f(ml[s * 2] - M);
    num = fmaf(w, pa[(size_t)s * D + d], num);
    den = fmaf(w, ml[s * 2 + 1], den);
  }
  Elem<T>::store(static_cast<T*>(a.out) + (size_t)bh * D + d, num / den);
}

template <class T, int D, int R>
cudaError_t run_decode(const DecodeArgs& a, cudaStream_t s) {
  constexpr int RG = D / Elem<T>::per16;
  constexpr int NG = kThreads / RG;
  constexpr size_t smem = sizeof(float) * NG * R * (D + 2);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<T, D, R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(a.splits, a.Hq / R, a.B);
  decode_kernel<T, D, R><<<grid, kThreads, smem, s>>>(a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (a.splits > 1) {
    decode_combine_kernel<T, D><<<a.B * a.Hq, D, 0, s>>>(a);
    e = cudaGetLastError();
  }
  return e;
}

template <class T, int D>
cudaError_t pick_r(const DecodeArgs& a, cudaStream_t s) {
  const int rep = a.Hq / a.Hkv;
  if (rep % 8 == 0) return run_decode<T, D, 8>(a, s);
  if (rep % 4 == 0) return run_decode<T, D, 4>(a, s);
  if (rep % 2 == 0) return run_decode<T, D, 2>(a, s);
  return run_decode<T, D, 1>(a, s);
}

}  // namespace

cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t s) {
  if (a.dtype == PYR_F32) return a.D == 64 ? pick_r<float, 64>(a, s) : pick_r<float, 128>(a, s);
  return a.D == 64 ? pick_r<__nv_bfloat16, 64>(a, s) : pick_r<__nv_bfloat16, 128>(a, s);
}

}  // namespace pyr
