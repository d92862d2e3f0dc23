// y[M, N] = x[M, K] . w[N, K]^T (+ residual) for bf16 with at most 64 rows of x: the linear layers of a
// decode step, where the weights are read once and everything else is small. Streaming the weights is
// the whole cost, so the kernel is shaped for bytes in flight, not for math:
//
//   * a CTA owns 128 output features and one slice of K; the slices of one feature block form a
//     thread-block cluster (1 to 8 CTAs), so a [4096 x 4096] weight becomes 256 independent streams,
//     two CTAs to an SM;
//   * the weights are the A operand (128 features = the 128 lanes of the accumulator), the rows of x
//     the B operand (64 columns of tensor memory): one elected thread feeds a four-stage ring of
//     [128 x 64] weight tiles and [64 x 64] x tiles by TMA, another issues 128 x 64 x 16 tcgen05 MMAs;
//   * every CTA re-reads x from L2, and CTAs launched together move in step: each starts its walk
//     over the K tiles at its own offset, so that at any moment the machine asks L2 for many
//     different lines of x rather than for the same few (the walk is fixed per CTA: results stay
//     bit-reproducible);
//   * the cluster adds its partial sums through distributed shared memory in slice order 0, 1, ... -
//     a fixed order, so the result does not depend on scheduling - and each CTA of the cluster
//     finishes (sum, residual, store) its own share of the tile's 64 rows.
//
// Rows of x beyond M are zero-filled by the tensor map and never stored. Every wait is bounded; a
// CTA whose wait ran out still takes part in the cluster's barriers.
#include <cuda_bf16.h>
#include <stddef.h>

#include "pyr_internal.h"
#include "tc_common.cuh"

namespace pyr {
namespace {

using namespace tc;

constexpr int kSkM = 64, kSkN = 128, kSkK = 64, kSkStages = 4, kSkThreads = 6 * 32;
constexpr int kSkWBytes = kSkN * kSkK * 2, kSkXBytes = kSkM * kSkK * 2;      // 16 KB + 8 KB per stage
constexpr int kRedStride = kSkN + 4;                                        // floats per row of the partial sums

struct SkSmem {
  alignas(1024) uint8_t w[kSkStages][kSkWBytes];
  alignas(1024) uint8_t x[kSkStages][kSkXBytes];
  uint64_t full[kSkStages], empty[kSkStages], acc_full;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(kSkM * kRedStride * 4 <= kSkStages * kSkWBytes, "partial sums reuse the weight ring");
static_assert(2 * (sizeof(SkSmem) + 1024 + 1024) <= 228 * 1024, "two CTAs per SM");

constexpr int kSkMaxParts = 4;

struct SkinnyArgs {
  const __nv_bfloat16* res;
  __nv_bfloat16* y[kSkMaxParts];   // the output's column parts, each [M, part_n] (one part: the whole of y)
  int part_n;
  int M, N, K, ktiles;      // ktiles = [64-wide] K tiles in all; slice i takes [i ktiles / slices, (i + 1) ktiles / slices)
  int* status;              // may be null
};

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
  return v;
}

__global__ void __launch_bounds__(kSkThreads, 2)
gemm_skinny_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, SkinnyArgs a) {
  extern __shared__ uint8_t sk_smem_raw[];
  SkSmem& sm = *reinterpret_cast<SkSmem*>((reinterpret_cast<uintptr_t>(sk_smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kSkN;
  const int slice = blockIdx.y, slices = gridDim.y;            // the cluster spans gridDim.y
  const int kt_begin = (int)((long long)slice * a.ktiles / slices);
  const int nkt = (int)((long long)(slice + 1) * a.ktiles / slices) - kt_begin;
  const int kt_rot = (int)((blockIdx.x * 3u) % (unsigned)nkt);
  volatile int* abort_flag = &sm.abort_flag;
  const int code = PYR_ERR_TIMEOUT;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kSkStages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
    mbar_init(&sm.acc_full, 1);
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 5) {
    tmem_alloc(&sm.tmem_base, kSkM);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 4) {
    if (lane == 0) {
      prefetch_tensormap(&map_x);
      prefetch_tensormap(&map_w);
      bool ok = true;
      for (int i = 0; i < nkt && ok; ++i) {
        const int st = i % kSkStages;
        if (i >= kSkStages) ok = mbar_wait(&sm.empty[st], ((i / kSkStages) - 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        int kt = kt_rot + i;
        if (kt >= nkt) kt -= nkt;
        const int k0 = (kt_begin + kt) * kSkK;
        mbar_expect_tx(&sm.full[st], kSkWBytes + kSkXBytes);
        tma_load_4d(sm.w[st], &map_w, &sm.full[st], k0, 0, n0, 0);
        tma_load_4d(sm.x[st], &map_x, &sm.full[st], k0, 0, 0, 0);
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(kSkN, kSkM, false, false);
      const uint64_t dw0 = smem_desc_sw128(smem_u32(sm.w[0]), 16, 1024), dx0 = smem_desc_sw128(smem_u32(sm.x[0]), 16, 1024);
      bool ok = true;
      for (int i = 0; i < nkt && ok; ++i) {
        const int st = i % kSkStages;
        ok = mbar_wait(&sm.full[st], (i / kSkStages) & 1, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        const uint64_t dw = dw0 + (uint64_t)((st * kSkWBytes) >> 4), dx = dx0 + (uint64_t)((st * kSkXBytes) >> 4);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ss(tmem, dw + (uint64_t)((kk * 32) >> 4), dx + (uint64_t)((kk * 32) >> 4), idesc, (i > 0 || kk > 0) ? 1u : 0u);
        mma_commit(&sm.empty[st]);
      }
      if (ok) mma_commit(&sm.acc_full);
    }
    __syncwarp();
  } else {
    // thread = feature n0 + threadIdx.x: its 64 partial sums (one per row of x) go to red[row][feature].
    // The accumulator's barrier fires when every MMA has read its tiles, so the weight ring is free.
    bool ok = mbar_wait(&sm.acc_full, 0, abort_flag, a.status, code);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      float* red = reinterpret_cast<float*>(&sm.w[0][0]);
      const uint32_t t_base = tmem + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
      for (int c32 = 0; c32 < kSkM / 32; ++c32) {
        uint32_t v[32];
        tmem_ld32(t_base + c32 * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) red[(c32 * 32 + e) * kRedStride + threadIdx.x] = __uint_as_float(v[e]);
      }
    }
  }
  tc_fence_before();
  if (slices > 1) cluster_sync_all(); else __syncthreads();

  // CTA `slice` finishes its share of the 64 rows: sums the slices in order, adds the residual, stores
  if (*abort_flag == 0) {
    const uint32_t red0 = smem_u32(&sm.w[0][0]);
    const float* red = reinterpret_cast<const float*>(&sm.w[0][0]);
    const int rows_per = (kSkM + slices - 1) / slices;
    for (int e = threadIdx.x; e < rows_per * (kSkN / 4); e += kSkThreads) {
      const int r = slice * rows_per + e / (kSkN / 4), c4 = (e % (kSkN / 4)) * 4;
      if (r >= a.M || r >= kSkM) continue;
      float4 v;
      if (slices > 1) {
        const uint32_t addr = red0 + (uint32_t)((r * kRedStride + c4) * 4);
        v = ld_cluster_f4(addr, 0);
        for (int s = 1; s < slices; ++s) {
          const float4 u = ld_cluster_f4(addr, (uint32_t)s);
          v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
        }
      } else {
        v = *reinterpret_cast<const float4*>(&red[r * kRedStride + c4]);
      }
      const int part = n0 / a.part_n;                        // a feature block lies within one part (part_n % 128 == 0)
      const int64_t o = (int64_t)r * a.part_n + (n0 - part * a.part_n) + c4;
      if (a.res) {
        const uint2 rr = *reinterpret_cast<const uint2*>(a.res + o);
        v.x += __uint_as_float(rr.x << 16); v.y += __uint_as_float(rr.x & 0xffff0000u);
        v.z += __uint_as_float(rr.y << 16); v.w += __uint_as_float(rr.y & 0xffff0000u);
      }
      uint2 ov;
      ov.x = pack_bf16(v.x, v.y);
      ov.y = pack_bf16(v.z, v.w);
      *reinterpret_cast<uint2*>(a.y[part] + o) = ov;
    }
  }
  if (slices > 1) cluster_sync_all(); else __syncthreads();     // peers may still be reading this CTA's partial sums
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, kSkM);
  }
}

// K slices per feature block: as many (up to the portable cluster size) as keep the grid on the machine at once
// (two CTAs per SM), each with at least four K tiles. A cluster lives inside one GPC and the GPCs' SM counts do
// not divide evenly, so the last few of the 2 x SMs places cannot all be filled by clusters: with 288 CTAs in
// clusters of three a second round of CTAs cost 13 % (35.0 vs 31.0 us on a 12288 x 4096 weight), hence the slack.
int skinny_slices(int N, int K, int sms) {
  const int tiles = N / kSkN, kt = K / kSkK;
  const int places = 2 * sms * 93 / 100;
  int s = places / tiles;
  if (s > 8) s = 8;
  while (s > 1 && kt / s < 4) --s;
  return s < 1 ? 1 : s;
}

}  // namespace

bool gemm_skinny_supported(const void* x, const void* w, const void* res, const void* y, int64_t M, int N, int K) {
  const uintptr_t al = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(y) |
                       reinterpret_cast<uintptr_t>(res);
  return tensor_maps_available() && al % 16 == 0 && M >= 1 && M <= kSkM && N % kSkN == 0 && K % kSkK == 0;
}

cudaError_t launch_gemm_skinny(const void* x, const void* w, const void* res, void* const* ys, int n_parts, int64_t M, int N,
                               int K, int* status, cudaStream_t s) {
  if (n_parts < 1 || n_parts > kSkMaxParts || N % n_parts || (n_parts > 1 && ((N / n_parts) % kSkN || res)))
    return cudaErrorInvalidValue;
  const int sms = device_sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const int smem = (int)sizeof(SkSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(gemm_skinny_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  CUtensorMap mx, mw;
  if (!make_tensor_map_bf16(&mx, x, 1, (int)M, 1, K, (int64_t)M * K, K, K, kSkM) ||
      !make_tensor_map_bf16(&mw, w, 1, N, 1, K, (int64_t)N * K, K, K, kSkN))
    return cudaErrorInvalidValue;
  const int slices = skinny_slices(N, K, sms);
  SkinnyArgs a;
  a.res = static_cast<const __nv_bfloat16*>(res);
  for (int i = 0; i < kSkMaxParts; ++i) a.y[i] = static_cast<__nv_bfloat16*>(ys[i < n_parts ? i : 0]);
  a.part_n = N / n_parts;
  a.M = (int)M; a.N = N; a.K = K; a.ktiles = K / kSkK; a.status = status;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(N / kSkN, slices, 1);
  cfg.blockDim = dim3(kSkThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = slices; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_skinny_kernel, mx, mw, a);
}

}  // namespace pyr
