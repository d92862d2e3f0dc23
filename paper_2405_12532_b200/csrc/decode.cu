// Generation-phase attention over one layer's compressed cache (Section 4.1:
// the generation phase reuses the smaller initial KV cache). One new query per
// (sequence, head) streams the layer's K and V once, so the kernel is bound by
// HBM bandwidth. Rows are split across CTAs (split-K); inside a CTA one
// producer thread keeps a ring of bulk copies (cp.async.bulk, 8 KB of K and
// 8 KB of V per stage) in flight while eight consumer warps reduce the stages
// that have landed in shared memory.
#include <cuda_bf16.h>

#include "pyr_internal.h"
#include "tc_common.cuh"

namespace pyr {
namespace {

using namespace tc;

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kConsumers = 256;            // 8 consumer warps
constexpr int kThreads = kConsumers + 32;  // + 1 producer warp
constexpr int kStages = 6;
constexpr int kChunkBytes = 8192;          // of K (and of V) per stage

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

struct DecodeSmem {
  alignas(128) uint8_t k[kStages][kChunkBytes];
  alignas(128) uint8_t v[kStages][kChunkBytes];
  uint64_t full[kStages], empty[kStages];
  int abort_flag;
};

// Online-softmax update of one head's state with U rows whose scores are s[u].
template <int U, int EPL>
__device__ __forceinline__ void absorb(float& m, float& l, float* acc, const float* s, const float (*vf)[EPL]) {
  float mx = s[0];
#pragma unroll
  for (int u = 1; u < U; ++u) mx = fmaxf(mx, s[u]);
  const float m_new = fmaxf(m, mx);
  const float corr = exp2f(m - m_new);
  float p[U], ps = 0.f;
#pragma unroll
  for (int u = 0; u < U; ++u) { p[u] = exp2f(s[u] - m_new); ps += p[u]; }
  l = l * corr + ps;
  m = m_new;
#pragma unroll
  for (int e = 0; e < EPL; ++e) {
    float x = acc[e] * corr;
#pragma unroll
    for (int u = 0; u < U; ++u) x = fmaf(p[u], vf[u][e], x);
    acc[e] = x;
  }
}

// grid (splits, Hq / R, B). A CTA serves R consecutive query heads that share
// one KV head over the rows [start, end) of that head's cache; the appended
// row (index len) comes straight from k_new / v_new. RG = lanes per cache row
// (16 bytes each); the 256 consumer threads form NG = 256 / RG row groups and a
// stage holds 2 * NG rows, two per group.
template <class T, int D, int R>
__global__ void __launch_bounds__(kThreads) decode_kernel(DecodeArgs a) {
  constexpr int EPL = Elem<T>::per16;
  constexpr int RG = D / EPL;
  constexpr int NG = kConsumers / RG;
  constexpr int U = 2;
  constexpr int CH = U * NG;                       // rows per stage
  constexpr int row_bytes = D * (int)sizeof(T);
  static_assert(CH * row_bytes == kChunkBytes, "stage size");
  extern __shared__ uint8_t smem_raw[];
  DecodeSmem& sm = *reinterpret_cast<DecodeSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  float* red = reinterpret_cast<float*>(sm.k);     // [NG][R][D + 2], reused once the ring has drained

  const int split = blockIdx.x, hy = blockIdx.y, b = blockIdx.z;
  const int h0 = hy * R;
  const int rep = a.Hq / a.Hkv;
  const int g = h0 / rep;
  const int t = threadIdx.x;
  const int total = a.len + 1;
  const int start = split * a.rows_per_split;
  const int end = min(start + a.rows_per_split, total);
  const int end_cached = min(end, a.len);          // rows below this come from the cache
  const int ncached = max(end_cached - start, 0);
  const int nchunks = (ncached + CH - 1) / CH;

  char* kc = static_cast<char*>(a.kc) + ((size_t)b * a.Hkv + g) * a.cap * row_bytes;
  char* vc = static_cast<char*>(a.vc) + ((size_t)b * a.Hkv + g) * a.cap * row_bytes;
  volatile int* abort_flag = &sm.abort_flag;

  if (t == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.empty[i], kConsumers / 32);
    }
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();

  if (t >= kConsumers) {
    // ------------------------------------------------------------ producer
    if (t == kConsumers) {
      bool ok = true;
      for (int c = 0; c < nchunks && ok; ++c) {
        const int st = c % kStages;
        if (c >= kStages) ok = mbar_wait(&sm.empty[st], ((c / kStages) - 1) & 1, abort_flag, a.status, PYR_ERR_TIMEOUT);
        if (!ok) break;
        const int row = start + c * CH;
        const uint32_t bytes = (uint32_t)min(CH, end_cached - row) * row_bytes;
        mbar_expect_tx(&sm.full[st], 2 * bytes);
        bulk_load(sm.k[st], kc + (size_t)row * row_bytes, bytes, &sm.full[st]);
        bulk_load(sm.v[st], vc + (size_t)row * row_bytes, bytes, &sm.full[st]);
      }
    }
  } else {
    // ------------------------------------------------------------ consumers
    const int grp = t / RG, ln = t % RG;
    const unsigned gmask = RG == 32 ? 0xffffffffu : (((1u << (RG % 32)) - 1u) << ((t % 32) / RG * RG));
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

    bool ok = true;
    for (int c = 0; c < nchunks && ok; ++c) {
      const int st = c % kStages;
      ok = mbar_wait(&sm.full[st], (c / kStages) & 1, abort_flag, a.status, PYR_ERR_TIMEOUT);
      if (!ok) break;
      const int rows_here = min(CH, ncached - c * CH);
      float kf[U][EPL], vf[U][EPL];
      bool valid[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int rr = u * NG + grp;
        valid[u] = rr < rows_here;
        uint4 kr = make_uint4(0, 0, 0, 0), vr = make_uint4(0, 0, 0, 0);
        if (valid[u]) {
          kr = *reinterpret_cast<const uint4*>(sm.k[st] + rr * row_bytes + ln * 16);
          vr = *reinterpret_cast<const uint4*>(sm.v[st] + rr * row_bytes + ln * 16);
        }
        Elem<T>::unpack(kr, kf[u]);
        Elem<T>::unpack(vr, vf[u]);
      }
      __syncwarp();
      if ((t & 31) == 0) mbar_arrive(&sm.empty[st]);     // this warp holds its rows in registers
      if (valid[0]) {                                     // uniform over the row group
#pragma unroll
        for (int r = 0; r < R; ++r) {
          float s[U];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            float d = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) d = fmaf(q[r][e], kf[u][e], d);
#pragma unroll
            for (int o = RG / 2; o > 0; o >>= 1) d += __shfl_xor_sync(gmask, d, o);
            s[u] = valid[u] ? d : -INFINITY;
          }
          absorb<U, EPL>(m[r], l[r], acc[r], s, vf);
        }
      }
    }

    // the appended row: read from k_new / v_new by row group 0, stored into the cache by
    // the first head group of this KV head
    if (ok && end > a.len && grp == 0) {
      const char* kn = static_cast<const char*>(a.k_new) + ((size_t)b * a.Hkv + g) * row_bytes;
      const char* vn = static_cast<const char*>(a.v_new) + ((size_t)b * a.Hkv + g) * row_bytes;
      const uint4 kr = *reinterpret_cast<const uint4*>(kn + ln * 16);
      const uint4 vr = *reinterpret_cast<const uint4*>(vn + ln * 16);
      if (h0 == g * rep) {
        *reinterpret_cast<uint4*>(kc + (size_t)a.len * row_bytes + ln * 16) = kr;
        *reinterpret_cast<uint4*>(vc + (size_t)a.len * row_bytes + ln * 16) = vr;
      }
      float kf[1][EPL], vf[1][EPL];
      Elem<T>::unpack(kr, kf[0]);
      Elem<T>::unpack(vr, vf[0]);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) d = fmaf(q[r][e], kf[0][e], d);
#pragma unroll
        for (int o = RG / 2; o > 0; o >>= 1) d += __shfl_xor_sync(gmask, d, o);
        float s[1] = {d};
        absorb<1, EPL>(m[r], l[r], acc[r], s, vf);
      }
    }

    // combine the NG row groups in a fixed order (the ring is idle: every stage was consumed)
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float* dst = red + ((size_t)grp * R + r) * (D + 2);
#pragma unroll
      for (int e = 0; e < EPL; ++e) dst[ln * EPL + e] = acc[r][e];
      if (ln == 0) { dst[D] = m[r]; dst[D + 1] = l[r]; }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
    if (!*abort_flag) {
      for (int o = t; o < R * D; o += kConsumers) {
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
  constexpr int NG = kConsumers / RG;
  static_assert(sizeof(float) * NG * R * (D + 2) <= sizeof(DecodeSmem::k) + sizeof(DecodeSmem::v),
                "reduction buffer fits in the rings");
  constexpr size_t smem = sizeof(DecodeSmem) + 128;
  cudaError_t e = cudaFuncSetAttribute(decode_kernel<T, D, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(a.splits, a.Hq / R, a.B);
  decode_kernel<T, D, R><<<grid, kThreads, smem, s>>>(a);
  e = cudaGetLastError();
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
