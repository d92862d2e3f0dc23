// tcgen05 kernels of the prefill step (bf16, head_dim 128).
//
// score_tc_kernel: Algorithm 1's "A_e <- weighted_avg(A[-L:, :-L], dim=-2)".
// With the softmax statistics (lse) of the L recent queries known, a CTA owns
// 128 context keys of one (sequence, selection group) and computes
// S^T = K_tile . Q_tile^T on the tensor cores with the keys on the TMEM lane
// axis. Each thread then owns one key and sums w_i * exp(s_ij - lse_i) over
// the recent queries i of every head of the group, in a fixed order. The
// L x c block of attention weights only ever exists as 128 x 128 tiles in
// tensor memory.
#include <cuda_bf16.h>

#include <mutex>

#include "pyr_internal.h"
#include "tc_common.cuh"

namespace pyr {

// ------------------------------------------------------------------ host: tensor maps
namespace {
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode = nullptr;
std::once_flag g_encode_once;

EncodeFn encode_fn() {
  std::call_once(g_encode_once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      g_encode = reinterpret_cast<EncodeFn>(fn);
  });
  return g_encode;
}
}  // namespace

bool make_tensor_map_bf16(CUtensorMap* map, const void* base, int B, int n, int H, int D, int64_t sb, int64_t sn,
                          int64_t sh, int box_rows) {
  EncodeFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)n, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)sh * 2, (cuuint64_t)sn * 2, (cuuint64_t)sb * 2};
  if (B == 1) strides[2] = strides[1] * (cuuint64_t)n;   // unused by any access; keep it a legal multiple of 16
  cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

namespace {

using namespace tc;

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kTile = 128;                 // keys per CTA, queries per step
constexpr int kHalfBytes = kTile * 128;    // one [128 rows x 64 bf16] swizzled half tile
constexpr int kTileBytes = 2 * kHalfBytes; // a [128 x 128] bf16 tile = two halves along D

enum TimeoutCode { kTimeoutScore = PYR_ERR_TIMEOUT };

// ------------------------------------------------------------------ score kernel
// Warps 0-3 and 4-7: two groups of 128 threads, thread = one key of the tile;
// group w takes the steps s with s % 2 == w and TMEM buffer w. Warp 8: one
// lane loads tiles by TMA and issues the MMAs.
constexpr int kScoreThreads = 288;

struct ScoreSmem {
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t q[2][kTileBytes];
  float bias[2][kTile];
  double partial[kTile];
  uint64_t ld_full[2], ld_empty[2], s_full[2], s_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kScoreThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, PrefillArgs a) {
  extern __shared__ uint8_t smem_raw[];
  ScoreSmem& sm = *reinterpret_cast<ScoreSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int tile = blockIdx.x, gsel = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = a.n, L = a.L, c = n - L;
  const int heads = a.Hq / a.G;
  const int rep = a.Hq / a.Hkv;
  const int nqt = (L + kTile - 1) / kTile;
  const int steps = heads * nqt;
  const int j0 = tile * kTile;
  volatile int* abort_flag = &sm.abort_flag;
  if (*reinterpret_cast<volatile int*>(a.status) != 0) return;   // an earlier CTA gave up: do not pile on

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.ld_full[i], 1);
      mbar_init(&sm.ld_empty[i], 1);
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.s_empty[i], kTile);
    }
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 8) {
    tmem_alloc(&sm.tmem_base, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 8) {
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      constexpr uint32_t idesc = idesc_bf16(kTile, kTile, false, false);
      int g_prev = -1, kslot = 1;
      // loads run one step ahead of the MMAs
      auto issue_loads = [&](int s, int& g_prev_io, int& kslot_io) {
        const int h = gsel * heads + s / nqt, qt = s % nqt, g = h / rep;
        const int st = s & 1;
        uint32_t bytes = kTileBytes;
        if (g != g_prev_io) { kslot_io ^= 1; bytes += kTileBytes; }
        mbar_expect_tx(&sm.ld_full[st], bytes);
        if (g != g_prev_io) {
          tma_load_4d(sm.k[kslot_io], &map_k, &sm.ld_full[st], 0, g, j0, b);
          tma_load_4d(sm.k[kslot_io] + kHalfBytes, &map_k, &sm.ld_full[st], 64, g, j0, b);
          g_prev_io = g;
        }
        tma_load_4d(sm.q[st], &map_q, &sm.ld_full[st], 0, h, c + qt * kTile, b);
        tma_load_4d(sm.q[st] + kHalfBytes, &map_q, &sm.ld_full[st], 64, h, c + qt * kTile, b);
      };
      int kslot_of_step[2] = {0, 0};
      issue_loads(0, g_prev, kslot);
      kslot_of_step[0] = kslot;
      bool ok = true;
      for (int s = 0; s < steps && ok; ++s) {
        const int st = s & 1;
        if (s + 1 < steps) {
          // the stage of step s+1 was read by the MMAs of step s-1
          if (s >= 1) ok = mbar_wait(&sm.ld_empty[(s + 1) & 1], ((s - 1) >> 1) & 1, abort_flag, a.status, kTimeoutScore);
          if (!ok) break;
          issue_loads(s + 1, g_prev, kslot);
          kslot_of_step[(s + 1) & 1] = kslot;
        }
        ok = mbar_wait(&sm.ld_full[st], (s >> 1) & 1, abort_flag, a.status, kTimeoutScore);
        if (!ok) break;
        if (s >= 2) ok = mbar_wait(&sm.s_empty[st], ((s - 2) >> 1) & 1, abort_flag, a.status, kTimeoutScore);
        if (!ok) break;
        tc_fence_after();
        const uint32_t ka = smem_u32(sm.k[kslot_of_step[st]]), qa = smem_u32(sm.q[st]);
        const uint32_t d_tmem = tmem + st * kTile;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
          mma_ss(d_tmem, smem_desc_sw128(ka + off, 16, 1024), smem_desc_sw128(qa + off, 16, 1024), idesc, kk > 0);
        }
        mma_commit(&sm.s_full[st]);
        mma_commit(&sm.ld_empty[st]);
      }
    }
    __syncwarp();
  } else {
    const int wg = warp >> 2;                 // 0 or 1
    const int key = threadIdx.x & (kTile - 1);
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const float sc2 = a.scale * kLog2e;
    double total = 0.0;
    bool ok = true;
    for (int s = wg; s < steps && ok; s += 2) {
      const int h = gsel * heads + s / nqt, qt = s % nqt;
      const int i = qt * kTile + key;          // this thread prepares the bias of recent query i
      // the bias buffer of this group is free: every thread passed the barrier below after its reads
      sm.bias[wg][key] = i < L ? log2f(a.w[i]) - a.lse[((int64_t)b * a.Hq + h) * n + c + i] * kLog2e : -INFINITY;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + wg), "r"(kTile) : "memory");
      ok = mbar_wait(&sm.s_full[wg], (s >> 1) & 1, abort_flag, a.status, kTimeoutScore);
      if (!ok) break;
      tc_fence_after();
      float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tmem_ld32(tmem + lane_base + wg * kTile + ch * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int col = 0; col < 32; ++col)
          part[col & 3] += ex2(fmaf(__uint_as_float(r[col]), sc2, sm.bias[wg][ch * 32 + col]));
      }
      tc_fence_before();
      mbar_arrive(&sm.s_empty[wg]);
      total += (double)((part[0] + part[1]) + (part[2] + part[3]));
      asm volatile("bar.sync %0, %1;" ::"r"(1 + wg), "r"(kTile) : "memory");
    }
    if (wg == 1) sm.partial[key] = total;
    asm volatile("bar.sync 3, 256;" ::: "memory");
    if (wg == 0 && j0 + key < c && !*abort_flag)
      a.score[((int64_t)b * a.G + gsel) * c + j0 + key] = (float)((total + sm.partial[key]) / (double)heads);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

}  // namespace

bool score_tc_supported(const PrefillArgs& a) {
  return a.dtype == PYR_BF16 && a.D == 128 && encode_fn() != nullptr;
}
bool tensor_maps_available() { return encode_fn() != nullptr; }

cudaError_t launch_score_tc(const PrefillArgs& a, cudaStream_t s) {
  const int c = a.n - a.L;
  if (c <= 0) return cudaSuccess;
  CUtensorMap mq, mk;
  if (!make_tensor_map_bf16(&mq, a.q, a.B, a.n, a.Hq, a.D, a.qsb, a.qsn, a.qsh, kTile) ||
      !make_tensor_map_bf16(&mk, a.k, a.B, a.n, a.Hkv, a.D, a.ksb, a.ksn, a.ksh, kTile))
    return cudaErrorInvalidValue;
  const size_t smem = sizeof(ScoreSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((c + kTile - 1) / kTile, a.G, a.B);
  score_tc_kernel<<<grid, kScoreThreads, smem, s>>>(mq, mk, a);
  return cudaGetLastError();
}

}  // namespace pyr
