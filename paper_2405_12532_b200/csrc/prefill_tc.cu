// tcgen05 kernels of the prefill step (bf16, head_dim 128).
//
// score_tc_kernel: Algorithm 1's "A_e <- weighted_avg(A[-L:, :-L], dim=-2)".
// With the softmax statistics (lse) of the L recent queries known, a CTA owns
// one (sequence, head): its recent queries stay in shared memory and the
// context keys stream through once. S^T = K_tile . Q_tile^T runs on the tensor
// cores with the keys on the TMEM lane axis, so a thread owns one key and sums
// w_i * exp(s_ij - lse_i) over the recent queries i. The L x c block of
// attention weights only ever exists as 128 x 128 tiles in tensor memory.
// score_reduce_kernel then adds the heads of a selection group in a fixed order.
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

// Dense [batch][heads][rows][128] bf16 (the layer caches), seen as 2 * rows half-rows of 64 elements so
// that one box of 2 * box_rows half-rows is box_rows whole rows, contiguous in memory:
// coordinates are (0, 2 * row, head, batch); half-row j lands at offset 128 j, 16-byte chunk c at c ^ (j & 7).
bool make_tensor_map_rows_bf16(CUtensorMap* map, const void* base, int batch, int heads, int rows, int box_rows) {
  EncodeFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t dims[4] = {64, (cuuint64_t)rows * 2, (cuuint64_t)heads, (cuuint64_t)batch};
  cuuint64_t strides[3] = {128, (cuuint64_t)rows * 256, (cuuint64_t)heads * rows * 256};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows * 2, 1, 1};
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
// Work item = one (sequence, head) and up to kMaxQTiles tiles of 128 recent
// queries, which stay in shared memory while the context keys of the head
// stream through once, 128 per tile. The grid is one CTA per SM; a CTA takes
// items blockIdx.x, blockIdx.x + gridDim.x, ... so the K ring keeps running
// from one item into the next (one lane of a loader warp issues the TMA loads).
// Per (key tile, query tile) step S^T = K_tile . Q_tile^T (keys on the TMEM lane
// axis) goes into one of four TMEM buffers; one lane each of two warps issues
// the even and the odd steps, because the waits, fences and commits around a
// step's eight MMAs cost an issuing thread almost as much time as the MMAs take
// and the pipe idles meanwhile (measured: 1450 clocks per step with one issuing
// thread against 512 of tensor work). Sixteen compute warps in four groups:
// group g takes the steps s with s % 4 == g (so the four warps that share a
// scheduler are always in different phases and the special-function unit stays
// busy); a thread owns one key and sums w_i * exp(s_ij - lse_i) over the 128
// query columns of its steps, then writes the key's partial score of
// (head, query chunk, group). A second kernel adds the partial scores of a
// selection group in a fixed order.
constexpr int kScoreGroups = 4;             // compute groups of four warps
constexpr int kScoreCompute = 4 * kScoreGroups;
constexpr int kScoreThreads = (kScoreCompute + 3) * 32;   // then: MMA issue (even steps), TMA loads, MMA issue (odd steps)
constexpr int kScoreBufs = 4;              // TMEM buffers of 128 columns
constexpr int kMaxQTiles = 4;              // query tiles resident per item
constexpr int kScoreTiles = 6;             // 32 KB tiles of shared memory: the query tiles, then the K stages

struct ScoreSmem {
  alignas(1024) uint8_t tiles[kScoreTiles][kTileBytes];
  alignas(16) float bias[2][kMaxQTiles * kTile];     // of this item / of the next one
  uint64_t q_full, q_empty, k_full[kScoreTiles], k_empty[kScoreTiles], s_full[kScoreBufs], s_empty[kScoreBufs];
  uint32_t tmem_base;
  int abort_flag;
};

struct ScoreItem {
  int b, h, chunk, q0, nq;
};

__global__ void __launch_bounds__(kScoreThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, PrefillArgs a,
                float* partial, int nchunk, int nitems) {
  extern __shared__ uint8_t smem_raw[];
  ScoreSmem& sm = *reinterpret_cast<ScoreSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = a.n, L = a.L, c = n - L;
  const int rep = a.Hq / a.Hkv;
  const int nq_max = min(kMaxQTiles, (L + kTile - 1) / kTile);
  const int kst = kScoreTiles - nq_max;                             // K stages (>= 2)
  const int nkt = (c + kTile - 1) / kTile;
  const int my_items = ((int)blockIdx.x < nitems) ? (nitems - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  auto item_of = [&](int k) {                                       // k-th item of this CTA; heads vary fastest
    const int id = blockIdx.x + k * gridDim.x;
    ScoreItem it;
    it.h = id % a.Hq;
    it.chunk = (id / a.Hq) % nchunk;
    it.b = id / (a.Hq * nchunk);
    it.q0 = it.chunk * kMaxQTiles * kTile;
    it.nq = min(kMaxQTiles, (L - it.q0 + kTile - 1) / kTile);
    return it;
  };
  volatile int* abort_flag = &sm.abort_flag;

  if (threadIdx.x == 0) {
    mbar_init(&sm.q_full, 1);
    mbar_init(&sm.q_empty, 2);                   // both issuing threads
    for (int i = 0; i < kScoreTiles; ++i) {
      mbar_init(&sm.k_full[i], 1);
      mbar_init(&sm.k_empty[i], 2);
    }
    for (int i = 0; i < kScoreBufs; ++i) {
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.s_empty[i], kTile);          // the group that reads the buffer
    }
    // an earlier CTA of this launch gave up: the whole CTA leaves together (decided by one thread)
    sm.abort_flag = *reinterpret_cast<volatile int*>(a.status) != 0 ? 2 : 0;
    fence_barrier_init();
  }
  __syncthreads();
  if (sm.abort_flag == 2) return;
  if (warp == kScoreCompute) {
    tmem_alloc(&sm.tmem_base, kScoreBufs * kTile);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == kScoreCompute + 1) {
    // ---------------------------------------------------------------- TMA loads
    if (lane == 0 && my_items > 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      bool ok = true;
      int r = 0;                                  // K tiles loaded so far, over all items of this CTA
      int st = 0, use = 0;                        // stage of tile r and how often that stage was filled before
      for (int k = 0; k < my_items && ok; ++k) {
        const ScoreItem it = item_of(k);
        // the query tiles are free once the previous item's last MMAs have run
        if (k >= 1) ok = mbar_wait(&sm.q_empty, (k - 1) & 1, abort_flag, a.status, kTimeoutScore);
        if (!ok) break;
        mbar_expect_tx(&sm.q_full, (uint32_t)it.nq * kTileBytes);
        for (int qt = 0; qt < it.nq; ++qt) {
          tma_load_4d(sm.tiles[qt], &map_q, &sm.q_full, 0, it.h, c + it.q0 + qt * kTile, it.b);
          tma_load_4d(sm.tiles[qt] + kHalfBytes, &map_q, &sm.q_full, 64, it.h, c + it.q0 + qt * kTile, it.b);
        }
        const int g = it.h / rep;
        for (int j = 0; j < nkt && ok; ++j, ++r) {
          if (use > 0) ok = mbar_wait(&sm.k_empty[st], (use - 1) & 1, abort_flag, a.status, kTimeoutScore);
          if (!ok) break;
          uint8_t* dst = sm.tiles[nq_max + st];
          mbar_expect_tx(&sm.k_full[st], kTileBytes);
          tma_load_4d(dst, &map_k, &sm.k_full[st], 0, g, j * kTile, it.b);
          tma_load_4d(dst + kHalfBytes, &map_k, &sm.k_full[st], 64, g, j * kTile, it.b);
          if (++st == kst) { st = 0; ++use; }
        }
      }
    }
    __syncwarp();
  } else if (warp == kScoreCompute || warp == kScoreCompute + 2) {
    // ---------------------------------------------------------------- MMA issue: steps of one parity
    if (lane == 0 && my_items > 0) {
      const int mine = warp == kScoreCompute ? 0 : 1;
      constexpr uint32_t idesc = idesc_bf16(kTile, kTile, false, false);
      bool ok = true;
      int s = 0;                 // step = (key tile, query tile), numbered across items
      int st = 0, use = 0;       // stage of the current K tile and how often it was filled before
      for (int k = 0; k < my_items && ok; ++k) {
        const ScoreItem it = item_of(k);
        ok = mbar_wait(&sm.q_full, k & 1, abort_flag, a.status, kTimeoutScore);
        bool any_in_item = false;
        for (int j = 0; j < nkt && ok; ++j) {
          ok = mbar_wait(&sm.k_full[st], use & 1, abort_flag, a.status, kTimeoutScore);
          const uint64_t kd = smem_desc_sw128(smem_u32(sm.tiles[nq_max + st]), 16, 1024);
          bool any = false;
          for (int qt = 0; qt < it.nq && ok; ++qt, ++s) {
            if ((s & 1) != mine) continue;
            const int buf = s & (kScoreBufs - 1);
            if (s >= kScoreBufs)
              ok = mbar_wait(&sm.s_empty[buf], ((s / kScoreBufs) - 1) & 1, abort_flag, a.status, kTimeoutScore);
            if (!ok) break;
            tc_fence_after();
            const uint64_t qd = smem_desc_sw128(smem_u32(sm.tiles[qt]), 16, 1024);
            const uint32_t d_tmem = tmem + buf * kTile;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
              mma_ss(d_tmem, kd + off, qd + off, idesc, kk > 0);
            }
            mma_commit(&sm.s_full[buf]);
            any = true;
          }
          if (!ok) break;
          // the stage is free when both threads are through with it: after its MMAs of this tile, or at once
          if (any) mma_commit(&sm.k_empty[st]);
          else mbar_arrive(&sm.k_empty[st]);
          any_in_item |= any;
          if (++st == kst) { st = 0; ++use; }
        }
        if (ok) {
          if (any_in_item) mma_commit(&sm.q_empty);
          else mbar_arrive(&sm.q_empty);
        }
      }
    }
    __syncwarp();
  } else {
    const int wg = warp >> 2;                 // takes the steps whose running number is wg modulo 4
    const int key = threadIdx.x & (kTile - 1);
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const float sc2 = a.scale * kLog2e;
    // bias of recent query i: log2 w_i - lse_i log2 e; -inf beyond the window (those Q rows are zero fill).
    // A thread fetches its (at most two) entries of the next item while it works on this one.
    auto bias_of = [&](const ScoreItem& it, int i) -> float {
      const int qi = it.q0 + i;
      return (i < it.nq * kTile && qi < L)
                 ? log2f(a.w[qi]) - a.lse[((int64_t)it.b * a.Hq + it.h) * n + c + qi] * kLog2e
                 : -INFINITY;
    };
    static_assert(kScoreGroups * kTile == kMaxQTiles * kTile, "one bias entry per compute thread");
    float nb = my_items > 0 ? bias_of(item_of(0), threadIdx.x) : 0.f;
    bool ok = true;
    int sg = 0;   // steps of earlier items
    for (int k = 0; k < my_items && ok; ++k) {
      const ScoreItem it = item_of(k);
      float* bias = sm.bias[k & 1];
      bias[threadIdx.x] = nb;
      // every thread is past its reads of this buffer (item k - 2) since it went through the barrier of item k - 1
      asm volatile("bar.sync 1, %0;" ::"n"(kScoreGroups * kTile) : "memory");
      if (k + 1 < my_items) nb = bias_of(item_of(k + 1), threadIdx.x);
      float* dst = partial + (((int64_t)it.b * a.Hq + it.h) * nchunk + it.chunk) * kScoreGroups * (int64_t)c + (int64_t)wg * c;
      const int nq = it.nq;
      const int steps = nkt * nq;
      double total = 0.0;
      int jacc = -1;     // key tile `total` belongs to
      // stores this group's share of key tiles jacc .. upto - 1 (zero where it had no step)
      auto flush = [&](int upto) {
        for (int j = jacc < 0 ? 0 : jacc; j < upto; ++j) {
          if (j * kTile + key < c) dst[j * kTile + key] = (j == jacc) ? (float)total : 0.f;
        }
        total = 0.0;
      };
      // 32 query columns at a time: the TMEM load of the next quarter is in flight during the
      // exponentials of this one (two register sets)
      auto weigh = [&](const uint32_t* r, const float* bias_cols) -> float {
        const float4* bias4 = reinterpret_cast<const float4*>(bias_cols);
        float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const float4 bv = bias4[c4];
          part[0] += ex2(fmaf(__uint_as_float(r[c4 * 4 + 0]), sc2, bv.x));
          part[1] += ex2(fmaf(__uint_as_float(r[c4 * 4 + 1]), sc2, bv.y));
          part[2] += ex2(fmaf(__uint_as_float(r[c4 * 4 + 2]), sc2, bv.z));
          part[3] += ex2(fmaf(__uint_as_float(r[c4 * 4 + 3]), sc2, bv.w));
        }
        return (part[0] + part[1]) + (part[2] + part[3]);
      };
      const int s0 = (wg - sg) & (kScoreGroups - 1);
      int j = s0 / nq, qt = s0 - j * nq;         // key tile and query tile of step s, kept without dividing again
      for (int s = s0; s < steps && ok; s += kScoreGroups, qt += kScoreGroups) {
        while (qt >= nq) { qt -= nq; ++j; }
        if (j != jacc) {
          flush(j);
          jacc = j;
        }
        const int buf = (sg + s) & (kScoreBufs - 1);
        ok = mbar_wait(&sm.s_full[buf], ((sg + s) / kScoreBufs) & 1, abort_flag, a.status, kTimeoutScore);
        if (!ok) break;
        tc_fence_after();
        const uint32_t t_addr = tmem + lane_base + buf * kTile;
        const float* bq = &bias[qt * kTile];
        uint32_t ra[32], rb[32];
        tmem_ld32(t_addr, ra);
        tmem_wait_ld();
        tmem_ld32(t_addr + 32, rb);
        float v = weigh(ra, bq);
        tmem_wait_ld();
        tmem_ld32(t_addr + 64, ra);
        v += weigh(rb, bq + 32);
        tmem_wait_ld();
        tmem_ld32(t_addr + 96, rb);
        v += weigh(ra, bq + 64);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(&sm.s_empty[buf]);            // the values are in registers: the buffer can be refilled
        v += weigh(rb, bq + 96);
        total += (double)v;
      }
      if (ok) flush(nkt);
      sg += steps;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kScoreCompute) {
    tc_fence_after();
    tmem_dealloc(tmem, kScoreBufs * kTile);
  }
}

// score[b, g, j] = mean over the heads of group g of their summed partial scores, added in a fixed order.
__global__ void score_reduce_kernel(const float* __restrict__ partial, float* __restrict__ score, int c, int G,
                                    int rows_per_group, int heads, const int* status) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int gsel = blockIdx.y, b = blockIdx.z;
  if (j >= c || *status != 0) return;
  const float* src = partial + ((int64_t)b * G + gsel) * rows_per_group * (int64_t)c + j;
  double acc = 0.0;
  for (int r = 0; r < rows_per_group; ++r) acc += (double)src[(int64_t)r * c];
  score[((int64_t)b * G + gsel) * c + j] = (float)(acc / (double)heads);
}

}  // namespace

bool score_tc_supported(const PrefillArgs& a) {
  return a.dtype == PYR_BF16 && a.D == 128 && encode_fn() != nullptr;
}
bool tensor_maps_available() { return encode_fn() != nullptr; }

int score_tc_groups() { return kScoreGroups; }
int score_tc_chunks(int L) { return ((L + kTile - 1) / kTile + kMaxQTiles - 1) / kMaxQTiles; }

cudaError_t launch_score_tc(const PrefillArgs& a, float* partial, cudaStream_t s) {
  const int c = a.n - a.L;
  if (c <= 0) return cudaSuccess;
  CUtensorMap mq, mk;
  if (!make_tensor_map_bf16(&mq, a.q, a.B, a.n, a.Hq, a.D, a.qsb, a.qsn, a.qsh, kTile) ||
      !make_tensor_map_bf16(&mk, a.k, a.B, a.n, a.Hkv, a.D, a.ksb, a.ksn, a.ksh, kTile))
    return cudaErrorInvalidValue;
  const size_t smem = sizeof(ScoreSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int nchunk = score_tc_chunks(a.L);
  const int nitems = a.B * nchunk * a.Hq;
  int dev = 0, sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int grid = nitems < sms ? nitems : sms;
  score_tc_kernel<<<grid, kScoreThreads, smem, s>>>(mq, mk, a, partial, nchunk, nitems);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int heads = a.Hq / a.G;
  dim3 rgrid((c + 255) / 256, a.G, a.B);
  score_reduce_kernel<<<rgrid, 256, 0, s>>>(partial, a.score, c, a.G, heads * nchunk * kScoreGroups, heads, a.status);
  return cudaGetLastError();
}

}  // namespace pyr
