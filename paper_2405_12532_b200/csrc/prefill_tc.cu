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

// ------------------------------------------------------------------ attention kernel
// Algorithm 1, "compute attention weights of KV", and the attention output.
//
// A CTA owns 256 consecutive query rows of one (sequence, head): two 128-row
// tiles that share every K and V tile it loads. Warps 0-3 and 4-7 are the
// softmax groups of tile 0 and 1 (thread = one query row), warp 8 issues the
// MMAs, warp 9 the TMA loads. Tensor memory (512 columns): S0 | S1 | O0 | O1,
// 128 fp32 columns each; P (bf16) overwrites the first 64 columns of its S.
// Per key tile j the MMA order is PV0(j), S0(j+1), PV1(j), S1(j+1), so one
// group's softmax overlaps the other's tensor work. The running maximum used
// in the exponent is only raised when the row maximum has grown by more than
// 2^8, which keeps rescaling of O (a TMEM round trip) rare; the final
// normalisation uses the same maximum, so the result is the exact softmax.
constexpr int kAttnThreads = 320;
constexpr float kRescaleStep = 8.0f;

struct AttnSmem {
  alignas(1024) uint8_t q[2][kTileBytes];
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t v[2][kTileBytes];
  uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], p_ready[2], o_done[2];
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, PrefillArgs a) {
  extern __shared__ uint8_t smem_raw[];
  AttnSmem& sm = *reinterpret_cast<AttnSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int pair = gridDim.x - 1 - blockIdx.x;     // longest rows first
  const int h = blockIdx.y, b = blockIdx.z;
  const int g = h / (a.Hq / a.Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = a.n;
  const int r0 = pair * 2 * kTile;
  const bool valid1 = r0 + kTile < n;
  const int nkt0 = 2 * pair + 1;                   // key tiles of query tile 0 (diagonal last)
  const int nkt1 = valid1 ? 2 * pair + 2 : 0;
  const int nkt = valid1 ? nkt1 : nkt0;
  volatile int* abort_flag = &sm.abort_flag;
  if (*reinterpret_cast<volatile int*>(a.status) != 0) return;

  if (threadIdx.x == 0) {
    mbar_init(&sm.q_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.k_full[i], 1);
      mbar_init(&sm.k_empty[i], 1);
      mbar_init(&sm.v_full[i], 1);
      mbar_init(&sm.v_empty[i], 1);
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.p_ready[i], kTile);
      mbar_init(&sm.o_done[i], 1);
    }
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 8) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const int code = PYR_ERR_TIMEOUT;

  if (warp == 9) {
    // ---------------------------------------------------------------- TMA loads
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      mbar_expect_tx(&sm.q_full, valid1 ? 2 * kTileBytes : kTileBytes);
      for (int w = 0; w < (valid1 ? 2 : 1); ++w) {
        tma_load_4d(sm.q[w], &map_q, &sm.q_full, 0, h, r0 + w * kTile, b);
        tma_load_4d(sm.q[w] + kHalfBytes, &map_q, &sm.q_full, 64, h, r0 + w * kTile, b);
      }
      bool ok = true;
      for (int j = 0; j < nkt && ok; ++j) {
        const int st = j & 1;
        if (j >= 2) ok = mbar_wait(&sm.k_empty[st], ((j - 2) >> 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        mbar_expect_tx(&sm.k_full[st], kTileBytes);
        tma_load_4d(sm.k[st], &map_k, &sm.k_full[st], 0, g, j * kTile, b);
        tma_load_4d(sm.k[st] + kHalfBytes, &map_k, &sm.k_full[st], 64, g, j * kTile, b);
        if (j >= 2) ok = mbar_wait(&sm.v_empty[st], ((j - 2) >> 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        mbar_expect_tx(&sm.v_full[st], kTileBytes);
        tma_load_4d(sm.v[st], &map_v, &sm.v_full[st], 0, g, j * kTile, b);
        tma_load_4d(sm.v[st] + kHalfBytes, &map_v, &sm.v_full[st], 64, g, j * kTile, b);
      }
    }
    __syncwarp();
  } else if (warp == 8) {
    // ---------------------------------------------------------------- MMA issue
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(kTile, kTile, false, false);   // S = Q K^T, both K-major
      constexpr uint32_t idesc_o = idesc_bf16(kTile, kTile, false, true);    // O += P V, V is MN-major
      // operand descriptors are built once; a k-step only adds a constant to the start-address field
      const uint64_t dq0 = smem_desc_sw128(smem_u32(sm.q[0]), 16, 1024), dq1 = smem_desc_sw128(smem_u32(sm.q[1]), 16, 1024);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, 1024), dk1 = smem_desc_sw128(smem_u32(sm.k[1]), 16, 1024);
      const uint64_t dv0 = smem_desc_sw128(smem_u32(sm.v[0]), kHalfBytes, 1024);
      const uint64_t dv1 = smem_desc_sw128(smem_u32(sm.v[1]), kHalfBytes, 1024);
      auto issue_s = [&](int w, int st) {
        const uint64_t qd = w ? dq1 : dq0, kd = st ? dk1 : dk0;
        const uint32_t d_tmem = tmem + w * kTile;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
          mma_ss(d_tmem, qd + off, kd + off, idesc_s, kk > 0);
        }
        mma_commit(&sm.s_full[w]);
      };
      auto issue_pv = [&](int w, int st, bool accumulate) {
        const uint64_t vd = st ? dv1 : dv0;
        const uint32_t d_tmem = tmem + (2 + w) * kTile, p_tmem = tmem + w * kTile;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)   // 16 keys per step: 8 TMEM columns of P, 16 rows of V
          mma_ts(d_tmem, p_tmem + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), idesc_o, (accumulate || kk > 0) ? 1u : 0u);
        mma_commit(&sm.o_done[w]);
      };
      bool ok = mbar_wait(&sm.q_full, 0, abort_flag, a.status, code);
      if (ok) ok = mbar_wait(&sm.k_full[0], 0, abort_flag, a.status, code);
      if (ok) {
        tc_fence_after();
        issue_s(0, 0);
        if (valid1) issue_s(1, 0);
        mma_commit(&sm.k_empty[0]);
      }
      for (int j = 0; j < nkt && ok; ++j) {
        const int st = j & 1, st1 = (j + 1) & 1;
        ok = mbar_wait(&sm.v_full[st], (j >> 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        bool k_next_ready = false;
        const int last_w = valid1 ? 1 : 0;
        for (int w = 0; w < 2 && ok; ++w) {
          const int nkt_w = w ? nkt1 : nkt0;
          if (j < nkt_w) {
            ok = mbar_wait(&sm.p_ready[w], j & 1, abort_flag, a.status, code);
            if (!ok) break;
            tc_fence_after();
            issue_pv(w, st, j > 0);
          }
          if (w == last_w) mma_commit(&sm.v_empty[st]);
          if (j + 1 < nkt_w) {
            if (!k_next_ready) {
              ok = mbar_wait(&sm.k_full[st1], ((j + 1) >> 1) & 1, abort_flag, a.status, code);
              if (!ok) break;
              k_next_ready = true;
              tc_fence_after();
            }
            issue_s(w, st1);
          }
          if (w == last_w && j + 1 < nkt) mma_commit(&sm.k_empty[st1]);
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- softmax groups
    const int w = warp >> 2;
    const int row_in_tile = threadIdx.x & (kTile - 1);
    const int i = r0 + w * kTile + row_in_tile;           // query row of this thread
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_addr = tmem + lane_base + w * kTile;
    const uint32_t o_addr = tmem + lane_base + (2 + w) * kTile;
    const int nkt_w = w ? nkt1 : nkt0;
    const float sc2 = a.scale * kLog2e;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nkt_w && ok; ++j) {
      ok = mbar_wait(&sm.s_full[w], j & 1, abort_flag, a.status, code);
      if (!ok) break;
      tc_fence_after();
      const bool diag = j == nkt_w - 1;     // diagonal tile: key 128 j + col is visible iff col <= lim
      const int lim = i - j * kTile;
      // pass 1: the row maximum (S is read twice from tensor memory rather than held in 128 registers)
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t ra[32], rb[32];
        tmem_ld32(s_addr + half * 64, ra);
        tmem_ld32(s_addr + half * 64 + 32, rb);
        tmem_wait_ld();
        if (diag) {
#pragma unroll
          for (int col = 0; col < 32; ++col) {
            if (half * 64 + col > lim) ra[col] = 0xff800000u;
            if (half * 64 + 32 + col > lim) rb[col] = 0xff800000u;
          }
        }
#pragma unroll
        for (int col = 0; col < 32; col += 4) {
          mx0 = max3(mx0, __uint_as_float(ra[col]), __uint_as_float(ra[col + 1]));
          mx1 = max3(mx1, __uint_as_float(ra[col + 2]), __uint_as_float(ra[col + 3]));
          mx2 = max3(mx2, __uint_as_float(rb[col]), __uint_as_float(rb[col + 1]));
          mx3 = max3(mx3, __uint_as_float(rb[col + 2]), __uint_as_float(rb[col + 3]));
        }
      }
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sc2;
      const bool need = mx > m_used + kRescaleStep;      // also true on the first tile (m_used = -inf)
      if (j > 0 && __any_sync(0xffffffffu, need)) {
        // O of this tile must hold every PV issued so far before it is rescaled
        ok = mbar_wait(&sm.o_done[w], (j - 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        const float f = need ? ex2(m_used - mx) : 1.f;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t o[32];
          tmem_ld32(o_addr + ch * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int col = 0; col < 32; ++col) o[col] = __float_as_uint(__uint_as_float(o[col]) * f);
          tmem_st32(o_addr + ch * 32, o);
        }
        l *= f;
      }
      if (need) m_used = mx;
      // pass 2: P = exp2(S * scale - m), written over S as bf16, 32 columns at a time; the next
      // 32 columns are in flight while these are exponentiated
      float part[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t buf[2][32];
      tmem_ld32(s_addr, buf[0]);
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t* cur = buf[ch & 1];
        tmem_wait_ld();
        if (ch < 3) tmem_ld32(s_addr + (ch + 1) * 32, buf[(ch + 1) & 1]);
        if (diag) {
#pragma unroll
          for (int col = 0; col < 32; ++col)
            if (ch * 32 + col > lim) cur[col] = 0xff800000u;
        }
        uint32_t p[16];
#pragma unroll
        for (int c2 = 0; c2 < 16; ++c2) {
          const float p0 = ex2(fmaf(__uint_as_float(cur[2 * c2]), sc2, -m_used));
          const float p1 = ex2(fmaf(__uint_as_float(cur[2 * c2 + 1]), sc2, -m_used));
          part[c2 & 1] += p0;
          part[2 + (c2 & 1)] += p1;
          p[c2] = pack_bf16(p0, p1);
        }
        tmem_st16(s_addr + ch * 16, p);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&sm.p_ready[w]);
      l += (part[0] + part[1]) + (part[2] + part[3]);
    }
    if (ok && nkt_w > 0) ok = mbar_wait(&sm.o_done[w], (nkt_w - 1) & 1, abort_flag, a.status, code);
    if (ok && nkt_w > 0) {
      tc_fence_after();
      const float inv = 1.f / l;
      __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.out) + b * a.osb + h * a.osh + (int64_t)i * a.osn;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t o[32];
        tmem_ld32(o_addr + ch * 32, o);
        tmem_wait_ld();
        if (i < n) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(o[q4 * 8 + 0]) * inv, __uint_as_float(o[q4 * 8 + 1]) * inv);
            pk.y = pack_bf16(__uint_as_float(o[q4 * 8 + 2]) * inv, __uint_as_float(o[q4 * 8 + 3]) * inv);
            pk.z = pack_bf16(__uint_as_float(o[q4 * 8 + 4]) * inv, __uint_as_float(o[q4 * 8 + 5]) * inv);
            pk.w = pack_bf16(__uint_as_float(o[q4 * 8 + 6]) * inv, __uint_as_float(o[q4 * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(out + ch * 32 + q4 * 8) = pk;
          }
        }
      }
      if (i < n) a.lse[((int64_t)b * a.Hq + h) * n + i] = (m_used + log2f(l)) * 0.6931471805599453f;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

bool score_tc_supported(const PrefillArgs& a) {
  return a.dtype == PYR_BF16 && a.D == 128 && encode_fn() != nullptr;
}
bool prefill_tc_supported(const PrefillArgs& a) {
  return a.dtype == PYR_BF16 && a.D == 128 && encode_fn() != nullptr;
}

cudaError_t launch_prefill_tc(const PrefillArgs& a, cudaStream_t s) {
  CUtensorMap mq, mk, mv;
  if (!make_tensor_map_bf16(&mq, a.q, a.B, a.n, a.Hq, a.D, a.qsb, a.qsn, a.qsh, kTile) ||
      !make_tensor_map_bf16(&mk, a.k, a.B, a.n, a.Hkv, a.D, a.ksb, a.ksn, a.ksh, kTile) ||
      !make_tensor_map_bf16(&mv, a.v, a.B, a.n, a.Hkv, a.D, a.ksb, a.ksn, a.ksh, kTile))
    return cudaErrorInvalidValue;
  const size_t smem = sizeof(AttnSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((a.n + 2 * kTile - 1) / (2 * kTile), a.Hq, a.B);
  attn_tc_kernel<<<grid, kAttnThreads, smem, s>>>(mq, mk, mv, a);
  return cudaGetLastError();
}

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
