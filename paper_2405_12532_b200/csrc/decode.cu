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
  const uint32_t limit = a.spin_limit ? a.spin_limit : kSpinLimit;

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
      int issued = 0;                                  // chunks handed to the copy engine
      for (int c = 0; c < nchunks && ok; ++c, ++issued) {
        const int st = c % kStages;
        if (c >= kStages) ok = mbar_wait_limit(&sm.empty[st], ((c / kStages) - 1) & 1, limit, abort_flag, a.status, PYR_ERR_TIMEOUT);
        if (!ok) break;
        if (c == a.skip_chunk) continue;               // (test aid) this chunk never arrives
        const int row = start + c * CH;
        const uint32_t bytes = (uint32_t)min(CH, end_cached - row) * row_bytes;
        mbar_expect_tx(&sm.full[st], 2 * bytes);
        bulk_load(sm.k[st], kc + (size_t)row * row_bytes, bytes, &sm.full[st]);
        bulk_load(sm.v[st], vc + (size_t)row * row_bytes, bytes, &sm.full[st]);
      }
      if (*abort_flag) {
        // A wait ran out somewhere in the CTA: nobody may be left to consume the last copies. They
        // must have landed before the CTA gives its shared memory back, so wait for them here
        // (bounded, without recording anything more).
        volatile int none = 0;
        for (int c = max(issued - kStages, 0); c < issued; ++c)
          if (c != a.skip_chunk) mbar_wait_limit(&sm.full[c % kStages], (c / kStages) & 1, kSpinLimit, &none, nullptr, 0);
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
      ok = mbar_wait_limit(&sm.full[st], (c / kStages) & 1, limit, abort_flag, a.status, PYR_ERR_TIMEOUT);
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

// ------------------------------------------------------------------ grouped-query heads on the tensor cores
// With R >= 4 query heads per KV head the CUDA-core kernel above is bound by its multiply-adds
// (every cache row is used R times), not by HBM. Here the R queries of a KV head are the rows
// (padded to 16) of warp-level tensor-core MMAs: S = Q K^T over 32 cache rows at a time, online
// softmax on the accumulator fragments, P (bf16) reused as the A operand of O += P V. Each of the
// three consumer warps takes every third chunk and keeps its own (m, l, O); the states are merged
// at the end exactly as in the kernel above. With six stages, stage c % 6 is only ever read by
// warp c % 3, so every full/empty barrier has one waiter that follows it phase by phase. (A first
// version with four warps let a warp meet a barrier it had skipped a phase of; a parity wait is
// then ambiguous, a stage could be released early, and the producer's second expect_tx on a
// barrier whose phase was still open faulted the kernel once loads completed out of order.) Stages are [32 rows x 128] bf16
// tiles of K and of V, each one contiguous 8 KB TMA load (the rows are seen as half-rows of 128 bytes
// with the 128-byte swizzle, which leaves ldmatrix with two-way bank conflicts instead of eight-way).
constexpr int kMmaWarps = 3;
static_assert(kMmaWarps * 2 == 6, "two stages per consumer warp");
constexpr int kMmaThreads = (kMmaWarps + 1) * 32;
constexpr int kMmaStages = 2 * kMmaWarps;
constexpr int kMmaRows = 32;                       // cache rows per stage
constexpr int kMmaHalf = kMmaRows * 128;           // [32 rows x 64 bf16]

struct MmaSmem {
  alignas(1024) uint8_t k[kMmaStages][2 * kMmaHalf];
  alignas(1024) uint8_t v[kMmaStages][2 * kMmaHalf];
  uint64_t full[kMmaStages], empty[kMmaStages];
  int abort_flag;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A B, A = 16 x 16 with rows 8..15 zero (a_lo: k 0..7, a_hi: k 8..15 of the thread's row), B = 16 x 8
__device__ __forceinline__ void mma_16816(float* c, uint32_t a_lo, uint32_t a_hi, uint32_t b0, uint32_t b1) {
  const uint32_t zero = 0;
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a_lo), "r"(zero), "r"(a_hi), "r"(zero), "r"(b0), "r"(b1));
}

// grid (splits, Hq / R, B), as decode_kernel. bf16, D = 128.
template <int R>
__global__ void __launch_bounds__(kMmaThreads) decode_mma_kernel(const __grid_constant__ CUtensorMap map_k,
                                                                  const __grid_constant__ CUtensorMap map_v,
                                                                  DecodeArgs a) {
  constexpr int D = 128;
  constexpr int row_bytes = D * 2;
  constexpr int NS = kMmaWarps + 1;                 // states to merge: one per warp + the appended row
  extern __shared__ uint8_t smem_raw[];
  MmaSmem& sm = *reinterpret_cast<MmaSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* red = reinterpret_cast<float*>(sm.k);      // [NS][R][D + 2], used once the ring has drained

  const int split = blockIdx.x, hy = blockIdx.y, b = blockIdx.z;
  const int h0 = hy * R;
  const int rep = a.Hq / a.Hkv;
  const int g = h0 / rep;
  const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
  const int total = a.len + 1;
  const int start = split * a.rows_per_split;
  const int end = min(start + a.rows_per_split, total);
  const int end_cached = min(end, a.len);
  const int ncached = max(end_cached - start, 0);
  const int nchunks = (ncached + kMmaRows - 1) / kMmaRows;
  volatile int* abort_flag = &sm.abort_flag;

  if (t == 0) {
    for (int i = 0; i < kMmaStages; ++i) {
      mbar_init(&sm.full[i], 1);
      mbar_init(&sm.empty[i], 1);
    }
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();

  if (warp == kMmaWarps) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      bool ok = true;
      for (int c = 0; c < nchunks && ok; ++c) {
        const int st = c % kMmaStages;
        if (c >= kMmaStages) ok = mbar_wait(&sm.empty[st], ((c / kMmaStages) - 1) & 1, abort_flag, a.status, PYR_ERR_TIMEOUT);
        if (!ok) break;
        const int row = start + c * kMmaRows;       // rows past the cache's capacity are zero fill
        mbar_expect_tx(&sm.full[st], 4 * kMmaHalf);
        tma_load_4d(sm.k[st], &map_k, &sm.full[st], 0, 2 * row, g, b);   // 32 whole rows: 8 KB contiguous
        tma_load_4d(sm.v[st], &map_v, &sm.full[st], 0, 2 * row, g, b);
      }
    }
  } else {
    // ------------------------------------------------------------ consumers
    const int gq = lane >> 2, tq = lane & 3;        // fragment row (query) and column pair
    const float sc2 = a.scale * kLog2e;
    // A fragments of Q: row gq of the group (zero beyond R), d = 16 ks + 2 tq (+ 8)
    uint32_t qa[8][2];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = qa[ks][1] = 0;
      if (gq < R) {
        const char* qrow = static_cast<const char*>(a.q) + ((size_t)b * a.Hq + h0 + gq) * row_bytes;
        qa[ks][0] = *reinterpret_cast<const uint32_t*>(qrow + (ks * 16 + tq * 2) * 2);
        qa[ks][1] = *reinterpret_cast<const uint32_t*>(qrow + (ks * 16 + 8 + tq * 2) * 2);
      }
    }
    float m = -INFINITY, l = 0.f;                   // of row gq; l is this thread's share of the row sum
    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    // ldmatrix: lane supplies row (lane & 7) of matrix (lane >> 3)
    const int mi = lane >> 3, mr = lane & 7;
    // Byte offsets of this lane's ldmatrix rows inside a stage, without the 16-key step (4096 bytes).
    // A stage holds half-rows of 128 bytes: half-row j = 2 * key + (d >= 64), 16-byte chunk c at c ^ (j & 7).
    uint32_t koff[8], voff[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      // K (plain): matrices (keys 0-7, d lo) (keys 0-7, d hi) (keys 8-15, d lo) (keys 8-15, d hi) of k-step i
      koff[i] = (uint32_t)((2 * ((mi >> 1) * 8 + mr) + (i >> 2)) * 128 +
                           ((((i & 3) * 2 + (mi & 1)) ^ ((2 * mr + (i >> 2)) & 7)) << 4));
      // V (transposed): matrices (keys 0-7, d lo) (keys 8-15, d lo) (keys 0-7, d hi) (keys 8-15, d hi) of column pair i
      voff[i] = (uint32_t)((2 * ((mi & 1) * 8 + mr) + (i >> 2)) * 128 +
                           ((((i & 3) * 2 + (mi >> 1)) ^ ((2 * mr + (i >> 2)) & 7)) << 4));
    }

    bool ok = true;
    for (int c = warp; c < nchunks && ok; c += kMmaWarps) {
      const int st = c % kMmaStages;
      ok = mbar_wait(&sm.full[st], (c / kMmaStages) & 1, abort_flag, a.status, PYR_ERR_TIMEOUT);
      if (!ok) break;
      const int rows_here = min(kMmaRows, ncached - c * kMmaRows);
      const uint32_t kb = smem_u32(sm.k[st]), vb = smem_u32(sm.v[st]);
      if (rows_here < kMmaRows) {
        // rows past the end of this split hold other data (or nothing): their scores are masked
        // below, and their V must not reach the MMA as NaN or Inf
        for (int i = lane; i < (kMmaRows - rows_here) * 16; i += 32) {
          const int row = rows_here + (i >> 4), ch = i & 15;
          const int j = 2 * row + (ch >> 3);       // half-row
          *reinterpret_cast<uint4*>(sm.v[st] + j * 128 + (((ch & 7) ^ (j & 7)) << 4)) = make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
      }
      // S = Q K^T: 4 key tiles of 8
      float sc[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
      for (int kp = 0; kp < 2; ++kp) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t bf[4];
          ldsm_x4(kb + kp * 4096 + koff[ks], bf);
          mma_16816(sc[2 * kp], qa[ks][0], qa[ks][1], bf[0], bf[1]);
          mma_16816(sc[2 * kp + 1], qa[ks][0], qa[ks][1], bf[2], bf[3]);
        }
      }
      // online softmax of row gq over the 32 keys (this thread: keys 8 nt + 2 tq, + 1)
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          sc[nt][e] *= sc2;
          if (rows_here < kMmaRows && nt * 8 + tq * 2 + e >= rows_here) sc[nt][e] = -INFINITY;
          mx = fmaxf(mx, sc[nt][e]);
        }
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m, mx);             // finite: key 0 of a stage is always valid
      const float corr = ex2(m - m_new);
      float ps = 0.f;
      uint32_t pa[2][2];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const float p0 = ex2(sc[nt][0] - m_new), p1 = ex2(sc[nt][1] - m_new);
        ps += p0 + p1;
        pa[nt >> 1][nt & 1] = pack_bf16(p0, p1);
      }
      l = l * corr + ps;
      m = m_new;
      if (__any_sync(0xffffffffu, corr != 1.f)) {    // once the maxima have settled there is nothing to rescale
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) { o[nt][0] *= corr; o[nt][1] *= corr; }
      }
      // O += P V: 2 steps of 16 keys, 16 tiles of 8 output columns
#pragma unroll
      for (int kp = 0; kp < 2; ++kp) {
#pragma unroll
        for (int np = 0; np < 8; ++np) {
          uint32_t bf[4];
          ldsm_x4_trans(vb + kp * 4096 + voff[np], bf);
          mma_16816(o[2 * np], pa[kp][0], pa[kp][1], bf[0], bf[1]);
          mma_16816(o[2 * np + 1], pa[kp][0], pa[kp][1], bf[2], bf[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[st]);    // this warp is done reading the stage
    }

    // merge the warps' states and the appended row in a fixed order (the ring is idle by now)
    asm volatile("bar.sync 1, %0;" ::"n"(kMmaWarps * 32) : "memory");
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (gq < R) {
      float* dst = red + ((size_t)warp * R + gq) * (D + 2);
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
        dst[nt * 8 + tq * 2] = o[nt][0];
        dst[nt * 8 + tq * 2 + 1] = o[nt][1];
      }
      if (tq == 0) { dst[D] = m; dst[D + 1] = l; }
    }
    if (warp == 0) {
      // the appended row, straight from k_new / v_new: a state with one key; the first head group
      // of the KV head also stores it into the cache
      const bool has_new = ok && end > a.len;
      const char* kn = static_cast<const char*>(a.k_new) + ((size_t)b * a.Hkv + g) * row_bytes;
      const char* vn = static_cast<const char*>(a.v_new) + ((size_t)b * a.Hkv + g) * row_bytes;
      float kf[4] = {0.f, 0.f, 0.f, 0.f}, vf[4] = {0.f, 0.f, 0.f, 0.f};
      if (has_new) {
        const uint2 kr = *reinterpret_cast<const uint2*>(kn + lane * 8);
        const uint2 vr = *reinterpret_cast<const uint2*>(vn + lane * 8);
        if (h0 == g * rep) {
          char* kc = static_cast<char*>(a.kc) + (((size_t)b * a.Hkv + g) * a.cap + a.len) * row_bytes;
          char* vc = static_cast<char*>(a.vc) + (((size_t)b * a.Hkv + g) * a.cap + a.len) * row_bytes;
          *reinterpret_cast<uint2*>(kc + lane * 8) = kr;
          *reinterpret_cast<uint2*>(vc + lane * 8) = vr;
        }
        kf[0] = __uint_as_float(kr.x << 16); kf[1] = __uint_as_float(kr.x & 0xffff0000u);
        kf[2] = __uint_as_float(kr.y << 16); kf[3] = __uint_as_float(kr.y & 0xffff0000u);
        vf[0] = __uint_as_float(vr.x << 16); vf[1] = __uint_as_float(vr.x & 0xffff0000u);
        vf[2] = __uint_as_float(vr.y << 16); vf[3] = __uint_as_float(vr.y & 0xffff0000u);
      }
      for (int r = 0; r < R; ++r) {
        float* dst = red + ((size_t)kMmaWarps * R + r) * (D + 2);
        float d = 0.f;
        if (has_new) {
          const uint2 qr = *reinterpret_cast<const uint2*>(static_cast<const char*>(a.q) +
                                                           ((size_t)b * a.Hq + h0 + r) * row_bytes + lane * 8);
          d = __uint_as_float(qr.x << 16) * kf[0] + __uint_as_float(qr.x & 0xffff0000u) * kf[1] +
              __uint_as_float(qr.y << 16) * kf[2] + __uint_as_float(qr.y & 0xffff0000u) * kf[3];
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
#pragma unroll
        for (int e = 0; e < 4; ++e) dst[lane * 4 + e] = vf[e];
        if (lane == 0) { dst[D] = has_new ? d * sc2 : -INFINITY; dst[D + 1] = has_new ? 1.f : 0.f; }
      }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kMmaWarps * 32) : "memory");
    if (!*abort_flag) {
      for (int i = t; i < R * D; i += kMmaWarps * 32) {
        const int r = i / D, d = i % D;
        float M = -INFINITY;
        for (int gI = 0; gI < NS; ++gI) M = fmaxf(M, red[((size_t)gI * R + r) * (D + 2) + D]);
        float num = 0.f, den = 0.f;
        for (int gI = 0; gI < NS; ++gI) {
          const float* src = red + ((size_t)gI * R + r) * (D + 2);
          const float w = exp2f(src[D] - M);
          num = fmaf(w, src[d], num);
          den = fmaf(w, src[D + 1], den);
        }
        const int h = h0 + r;
        if (a.splits == 1) {
          static_cast<__nv_bfloat16*>(a.out)[((size_t)b * a.Hq + h) * D + d] = __float2bfloat16_rn(num / den);
        } else {
          const size_t pi = ((size_t)b * a.Hq + h) * a.splits + split;
          a.part_acc[pi * D + d] = num;
          if (d == 0) { a.part_ml[pi * 2] = M; a.part_ml[pi * 2 + 1] = den; }
        }
      }
    }
  }
}

template <int R>
cudaError_t run_decode_mma(const DecodeArgs& a, cudaStream_t s) {
  static_assert(sizeof(float) * (kMmaWarps + 1) * R * (128 + 2) <= sizeof(MmaSmem::k), "merge buffer fits in the K ring");
  CUtensorMap mk, mv;
  if (!make_tensor_map_rows_bf16(&mk, a.kc, a.B, a.Hkv, a.cap, kMmaRows) ||
      !make_tensor_map_rows_bf16(&mv, a.vc, a.B, a.Hkv, a.cap, kMmaRows))
    return cudaErrorInvalidValue;
  constexpr size_t smem = sizeof(MmaSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(a.splits, a.Hq / R, a.B);
  decode_mma_kernel<R><<<grid, kMmaThreads, smem, s>>>(mk, mv, a);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (a.splits > 1) {
    decode_combine_kernel<__nv_bfloat16, 128><<<a.B * a.Hq, 128, 0, s>>>(a);
    e = cudaGetLastError();
  }
  return e;
}

// the tensor-core kernel needs TMA (16-byte aligned caches) and at least 4 query heads per KV head
bool decode_mma_usable(const DecodeArgs& a) {
  const int rep = a.Hq / a.Hkv;
  return a.dtype == PYR_BF16 && a.D == 128 && rep % 4 == 0 && tensor_maps_available() &&
         (reinterpret_cast<uintptr_t>(a.kc) | reinterpret_cast<uintptr_t>(a.vc)) % 16 == 0;
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
  if (decode_mma_usable(a)) return (a.Hq / a.Hkv) % 8 == 0 ? run_decode_mma<8>(a, s) : run_decode_mma<4>(a, s);
  if (a.dtype == PYR_F32) return a.D == 64 ? pick_r<float, 64>(a, s) : pick_r<float, 128>(a, s);
  return a.D == 64 ? pick_r<__nv_bfloat16, 64>(a, s) : pick_r<__nv_bfloat16, 128>(a, s);
}

}  // namespace pyr
