// tcgen05 GEMM of the decoder glue: y[M, N] = x[M, K] . w[N, K]^T (+ residual), bf16 in, fp32
// accumulation in tensor memory, bf16 out. (Not from the paper: the linear layers of a whole-model
// workload, so that the 7B-shaped model runs on this library's kernels at tensor-core speed.)
//
// Persistent CTAs (one per SM) walk 128 x BN output tiles; BN = 256 for wide problems, 128 when M
// is small and more CTAs are worth more than a wider tile (decode: the weights stream once).
//   warps 0-3  epilogue: thread = output row; TMEM -> registers -> (+ residual) -> bf16 -> global
//   warp 4     TMA loads of the x and w tiles, 64 K-elements (one 128-byte swizzle atom) per stage
//   warp 5     issues the MMAs: 4 per stage, 128 x BN x 16, both operands K-major from shared memory
// Two accumulator buffers of BN columns: the epilogue of a tile overlaps the main loop of the next.
// Tiles are ordered so that the CTAs running at one time share a band of 16 row blocks of x and a
// few column blocks of w, which stay in L2. Every barrier is followed phase by phase by its waiter.
//
// The gated form (kGated) computes out = silu(x . wg^T) * (x . wu^T) in one pass: a 256-column tile is
// 128 rows of wg beside the same 128 rows of wu (two TMA boxes into one stage), the accumulator holds
// the gate in columns 0-127 and the up projection in 128-255, and the epilogue multiplies them, so
// neither projection is ever written out.
#include <cuda_bf16.h>
#include <stddef.h>

#include <mutex>

#include "pyr_internal.h"
#include "tc_common.cuh"

namespace pyr {
namespace {

using namespace tc;

constexpr int kBM = 128, kBK = 64;
constexpr int kGemmThreads = 6 * 32;
constexpr int kGroupM = 16;                   // row blocks per band

template <int BN> struct GemmCfg {
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kABytes = kBM * kBK * 2;          // 16 KB
  static constexpr int kBBytes = BN * kBK * 2;           // 32 or 16 KB
};

template <int BN>
struct GemmSmem {
  alignas(1024) uint8_t a[GemmCfg<BN>::kStages][GemmCfg<BN>::kABytes];
  alignas(1024) uint8_t b[GemmCfg<BN>::kStages][GemmCfg<BN>::kBBytes];
  uint64_t full[GemmCfg<BN>::kStages], empty[GemmCfg<BN>::kStages];
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

struct GemmArgs {
  const __nv_bfloat16* res;   // [M, N] or null
  __nv_bfloat16* y;           // [M, N]
  int64_t M;
  int N, K;
  int* status;                // may be null
  RowMap res_map;             // rows of `res` that the rows of y add (identity when its list is null)
};

__device__ __forceinline__ void tile_of(int tile, int mblocks, int nblocks, int* mb, int* nb) {
  const int band = tile / (kGroupM * nblocks);
  const int m0 = band * kGroupM;
  const int rows = min(kGroupM, mblocks - m0);
  const int in = tile - band * kGroupM * nblocks;
  *nb = in / rows;
  *mb = m0 + in % rows;
}

template <int BN, bool kGated>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_w2, GemmArgs a) {
  static_assert(!kGated || BN == 256, "the gated form pairs two 128-row boxes");
  constexpr int kOutCols = kGated ? BN / 2 : BN;       // output columns per tile
  using Cfg = GemmCfg<BN>;
  constexpr int S = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  GemmSmem<BN>& sm = *reinterpret_cast<GemmSmem<BN>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mblocks = (int)((a.M + kBM - 1) / kBM), nblocks = (a.N + kOutCols - 1) / kOutCols;
  const int tiles = mblocks * nblocks;
  const int ksteps = a.K / kBK;
  volatile int* abort_flag = &sm.abort_flag;
  const int code = PYR_ERR_TIMEOUT;

  if (threadIdx.x == 0) {
    for (int i = 0; i < S; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.acc_full[i], 1); mbar_init(&sm.acc_empty[i], kBM); }
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 5) {
    tmem_alloc(&sm.tmem_base, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 4) {
    // ---------------------------------------------------------------- TMA loads
    if (lane == 0) {
      prefetch_tensormap(&map_x);
      prefetch_tensormap(&map_w);
      if (kGated) prefetch_tensormap(&map_w2);
      bool ok = true;
      int it = 0;                                 // stages filled so far
      for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
        int mb, nb;
        tile_of(tile, mblocks, nblocks, &mb, &nb);
        for (int ks = 0; ks < ksteps && ok; ++ks, ++it) {
          const int st = it % S;
          if (it >= S) ok = mbar_wait(&sm.empty[st], ((it / S) - 1) & 1, abort_flag, a.status, code);
          if (!ok) break;
          mbar_expect_tx(&sm.full[st], Cfg::kABytes + Cfg::kBBytes);
          tma_load_4d(sm.a[st], &map_x, &sm.full[st], ks * kBK, 0, mb * kBM, 0);
          if (kGated) {
            tma_load_4d(sm.b[st], &map_w, &sm.full[st], ks * kBK, 0, nb * kOutCols, 0);
            tma_load_4d(sm.b[st] + Cfg::kBBytes / 2, &map_w2, &sm.full[st], ks * kBK, 0, nb * kOutCols, 0);
          } else {
            tma_load_4d(sm.b[st], &map_w, &sm.full[st], ks * kBK, 0, nb * BN, 0);
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMAs
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(kBM, BN, false, false);
      const uint64_t da0 = smem_desc_sw128(smem_u32(sm.a[0]), 16, 1024), db0 = smem_desc_sw128(smem_u32(sm.b[0]), 16, 1024);
      bool ok = true;
      int it = 0, tcount = 0;
      for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
        const int buf = tcount & 1;
        // the accumulator buffer is free once the epilogue of the tile two back has read it
        if (tcount >= 2) ok = mbar_wait(&sm.acc_empty[buf], ((tcount >> 1) - 1) & 1, abort_flag, a.status, code);
        for (int ks = 0; ks < ksteps && ok; ++ks, ++it) {
          const int st = it % S;
          ok = mbar_wait(&sm.full[st], (it / S) & 1, abort_flag, a.status, code);
          if (!ok) break;
          tc_fence_after();
          const uint64_t da = da0 + (uint64_t)((st * Cfg::kABytes) >> 4), db = db0 + (uint64_t)((st * Cfg::kBBytes) >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_ss(tmem + buf * BN, da + (uint64_t)((kk * 32) >> 4), db + (uint64_t)((kk * 32) >> 4), idesc,
                   (ks > 0 || kk > 0) ? 1u : 0u);
          mma_commit(&sm.empty[st]);
        }
        if (ok) mma_commit(&sm.acc_full[buf]);
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue, thread = output row
    const int row = threadIdx.x;                  // 0..127
    const uint32_t t_base = tmem + ((uint32_t)(warp * 32) << 16);
    bool ok = true;
    int tcount = 0;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
      int mb, nb;
      tile_of(tile, mblocks, nblocks, &mb, &nb);
      const int buf = tcount & 1;
      ok = mbar_wait(&sm.acc_full[buf], (tcount >> 1) & 1, abort_flag, a.status, code);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int64_t m = (int64_t)mb * kBM + row;
      const int n0 = nb * kOutCols;
#pragma unroll 1
      for (int c32 = 0; c32 < kOutCols / 32; ++c32) {
        uint32_t v[32];
        tmem_ld32(t_base + buf * BN + c32 * 32, v);
        if (kGated) {
          uint32_t u[32];
          tmem_ld32(t_base + buf * BN + kOutCols + c32 * 32, u);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float g = __uint_as_float(v[e]);
            v[e] = __float_as_uint(g / (1.f + __expf(-g)) * __uint_as_float(u[e]));
          }
        } else {
          tmem_wait_ld();
        }
        if (c32 == kOutCols / 32 - 1) {           // the buffer is in registers: the tile after next may use it
          tc_fence_before();
          mbar_arrive(&sm.acc_empty[buf]);
        }
        const int n = n0 + c32 * 32;
        if (m < a.M && n < a.N) {                 // N is a multiple of 8: whole 16-byte chunks are in or out
          __nv_bfloat16* yp = a.y + m * a.N + n;
          const __nv_bfloat16* rp = a.res ? a.res + a.res_map.source_row(m) * a.N + n : nullptr;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            if (n + ch * 8 < a.N) {
              float f[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[ch * 8 + e]);
              if (rp) {
                const uint4 r = *reinterpret_cast<const uint4*>(rp + ch * 8);
                const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  f[2 * e] += __uint_as_float(rw[e] << 16);
                  f[2 * e + 1] += __uint_as_float(rw[e] & 0xffff0000u);
                }
              }
              uint4 o;
              o.x = pack_bf16(f[0], f[1]); o.y = pack_bf16(f[2], f[3]); o.z = pack_bf16(f[4], f[5]); o.w = pack_bf16(f[6], f[7]);
              *reinterpret_cast<uint4*>(yp + ch * 8) = o;
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, 2 * BN);
  }
}

template <int BN, bool kGated>
cudaError_t run_gemm(const CUtensorMap& mx, const CUtensorMap& mw, const CUtensorMap& mw2, const GemmArgs& a, int sms,
                     cudaStream_t s) {
  const size_t smem = sizeof(GemmSmem<BN>) + 1024;
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, kGated>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int out_cols = kGated ? BN / 2 : BN;
  const long long tiles = ((a.M + kBM - 1) / kBM) * (long long)((a.N + out_cols - 1) / out_cols);
  const int grid = (int)(tiles < sms ? tiles : sms);
  gemm_tc_kernel<BN, kGated><<<grid, kGemmThreads, smem, s>>>(mx, mw, mw2, a);
  return cudaGetLastError();
}

// The glue calls have no cache handle, so the GEMMs' bounded waits report to a word of the library's own, one
// per GPU (a static device variable: nothing is allocated).
__device__ int g_glue_status = 0;
constexpr int kGlueMaxDevices = 64;
int* g_glue_status_ptr[kGlueMaxDevices] = {};
std::mutex g_glue_mutex;

}  // namespace

int* glue_status_word() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kGlueMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_glue_mutex);
  if (!g_glue_status_ptr[dev]) {
    int* w = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&w), g_glue_status) != cudaSuccess) return nullptr;
    g_glue_status_ptr[dev] = w;
  }
  return g_glue_status_ptr[dev];
}

bool gemm_tc_supported(const void* x, const void* w, const void* res, const void* y, int64_t M, int N, int K) {
  const uintptr_t al = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(y) |
                       reinterpret_cast<uintptr_t>(res);
  return tensor_maps_available() && al % 16 == 0 && K % kBK == 0 && N % 8 == 0 && M >= 1 && M < (1ll << 31) && N >= 8;
}

cudaError_t launch_gemm_tc(const void* x, const void* w, const void* res, void* y, int64_t M, int N, int K, int* status,
                           const RowMap& res_map, cudaStream_t s) {
  const int sms = device_sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  // wide tiles when there are enough of them to fill the machine, else narrower ones
  const long long tiles256 = ((M + kBM - 1) / kBM) * (long long)((N + 255) / 256);
  const int BN = tiles256 >= 2LL * sms ? 256 : 128;
  CUtensorMap mx, mw;
  if (!make_tensor_map_bf16(&mx, x, 1, (int)M, 1, K, (int64_t)M * K, K, K, kBM) ||
      !make_tensor_map_bf16(&mw, w, 1, N, 1, K, (int64_t)N * K, K, K, BN))
    return cudaErrorInvalidValue;
  GemmArgs a;
  a.res = static_cast<const __nv_bfloat16*>(res); a.y = static_cast<__nv_bfloat16*>(y);
  a.M = M; a.N = N; a.K = K; a.status = status; a.res_map = res_map;
  return BN == 256 ? run_gemm<256, false>(mx, mw, mw, a, sms, s) : run_gemm<128, false>(mx, mw, mw, a, sms, s);
}

// out[M, N] = silu(x . wg^T) * (x . wu^T): the gated form of the kernel above
cudaError_t launch_gemm_tc_gated(const void* x, const void* wg, const void* wu, void* out, int64_t M, int N, int K,
                                 int* status, cudaStream_t s) {
  const int sms = device_sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  CUtensorMap mx, mg, mu;
  if (!make_tensor_map_bf16(&mx, x, 1, (int)M, 1, K, (int64_t)M * K, K, K, kBM) ||
      !make_tensor_map_bf16(&mg, wg, 1, N, 1, K, (int64_t)N * K, K, K, 128) ||
      !make_tensor_map_bf16(&mu, wu, 1, N, 1, K, (int64_t)N * K, K, K, 128))
    return cudaErrorInvalidValue;
  GemmArgs a;
  a.res = nullptr; a.y = static_cast<__nv_bfloat16*>(out);
  a.M = M; a.N = N; a.K = K; a.status = status;
  return run_gemm<256, true>(mx, mg, mu, a, sms, s);
}

}  // namespace pyr
