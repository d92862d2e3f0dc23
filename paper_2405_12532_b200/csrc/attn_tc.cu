// tcgen05 causal attention of the prefill step (bf16, head_dim 128):
// Algorithm 1, "compute attention weights of KV", and the attention output.
//
// A CTA owns 256 consecutive query rows of one (sequence, head): two 128-row
// tiles that share every K and V tile it loads.
//   warps 0-15  softmax: tile w = warp / 8; the two warps that serve the same 32 rows
//               (warp % 4 = TMEM lane quarter) split the 128 keys of a tile in halves
//   warp 16     MMA issue for both tiles (one lane)
//   warp 17     TMA loads (one lane)
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; P
// (bf16) overwrites the first 64 columns of its S. Per tile and key tile j the
// order is S(j) -> softmax -> PV(j) -> S(j+1); the issuing thread alternates
// between the tiles (PV0 S0 PV1 S1), so one tile's softmax overlaps the
// other's tensor work. The running maximum used in the exponent is
// only raised when the row maximum has grown by more than 2^8, which keeps
// rescaling of O (a TMEM round trip) rare; the final normalisation uses the same
// maximum, so the result is the exact softmax.
#include <cuda_bf16.h>

#include "pyr_internal.h"
#include "tc_common.cuh"

namespace pyr {
namespace {

using namespace tc;

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTile = 128;
constexpr int kHalfBytes = kTile * 128;     // one [128 rows x 64 bf16] swizzled half tile
constexpr int kTileBytes = 2 * kHalfBytes;  // a [128 x 128] bf16 tile = two halves along D
constexpr int kSoftmaxWarps = 16;
constexpr int kThreads = (kSoftmaxWarps + 2) * 32;
constexpr float kRescaleStep = 8.0f;

struct AttnSmem {
  alignas(1024) uint8_t q[2][kTileBytes];
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t v[2][kTileBytes];
  float xmax[2][2][2][kTile];   // [tile][step parity][key half][row]
  float xsum[2][2][kTile];      // [tile][key half][row]
  uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], p_ready[2], o_done[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void pair_sync(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }
__device__ __forceinline__ void pair_arrive(int id) { asm volatile("bar.arrive %0, 64;" ::"r"(id) : "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
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
  const int users = valid1 ? 2 : 1;                // tiles that read each K / V stage
  volatile int* abort_flag = &sm.abort_flag;
  if (*reinterpret_cast<volatile int*>(a.status) != 0) return;   // an earlier CTA gave up: do not pile on

  if (threadIdx.x == 0) {
    mbar_init(&sm.q_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.k_full[i], 1);
      mbar_init(&sm.k_empty[i], 1);
      mbar_init(&sm.v_full[i], 1);
      mbar_init(&sm.v_empty[i], 1);
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.p_ready[i], 2 * kTile);
      mbar_init(&sm.o_done[i], 1);
    }
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kSoftmaxWarps) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const int code = PYR_ERR_TIMEOUT;

  if (warp == kSoftmaxWarps + 1) {
    // ---------------------------------------------------------------- TMA loads
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      mbar_expect_tx(&sm.q_full, users * kTileBytes);
      for (int w = 0; w < users; ++w) {
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
  } else if (warp >= kSoftmaxWarps) {
    // ---------------------------------------------------------------- MMA issue (one thread, both tiles)
    if (lane == 0 && warp == kSoftmaxWarps) {
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
      // Order per key tile j: PV0(j) S0(j+1) PV1(j) S1(j+1). While one tile's softmax runs, the
      // other tile's two groups keep the tensor pipe busy.
      bool ok = mbar_wait(&sm.q_full, 0, abort_flag, a.status, code);
      if (ok) ok = mbar_wait(&sm.k_full[0], 0, abort_flag, a.status, code);
      if (ok) {
        tc_fence_after();
        issue_s(0, 0);
        if (valid1) issue_s(1, 0);
        mma_commit(&sm.k_empty[0]);
      }
      const int last_w = valid1 ? 1 : 0;
      for (int j = 0; j < nkt && ok; ++j) {
        const int st = j & 1, st1 = (j + 1) & 1;
        ok = mbar_wait(&sm.v_full[st], (j >> 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        bool k_next_ready = false;
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
    // ---------------------------------------------------------------- softmax
    const int w = warp >> 3;                       // query tile
    const int hh = (warp >> 2) & 1;                // which 64 keys of a 128-key tile
    const int quarter = warp & 3;                  // TMEM lane quarter = rows 32 * quarter ...
    const int row = quarter * 32 + lane;
    const int i = r0 + w * kTile + row;            // query row of this thread
    const int bar_id = 1 + w * 4 + quarter;        // named barrier of the two warps that share these rows
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_addr = tmem + lane_base + w * kTile;            // S of the tile, column 0
    const uint32_t my_s = s_addr + hh * 64;                          // my 64 key columns
    const uint32_t my_p = s_addr + hh * 32;                          // where their bf16 P goes
    const uint32_t my_o = tmem + lane_base + (2 + w) * kTile + hh * 64;   // my 64 columns of O
    const int nkt_w = w ? nkt1 : nkt0;
    const float sc2 = a.scale * kLog2e;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nkt_w && ok; ++j) {
      ok = mbar_wait(&sm.s_full[w], j & 1, abort_flag, a.status, code);
      if (!ok) break;
      tc_fence_after();
      const bool diag = j == nkt_w - 1;            // diagonal tile: key 128 j + col is visible iff col <= lim
      const int lim = i - j * kTile - hh * 64;     // in my own column numbering
      // pass 1: maximum over my 64 keys, then over the partner's
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
      {
        uint32_t ra[32], rb[32];
        tmem_ld32(my_s, ra);
        tmem_ld32(my_s + 32, rb);
        tmem_wait_ld();
        if (diag) {
#pragma unroll
          for (int col = 0; col < 32; ++col) {
            if (col > lim) ra[col] = 0xff800000u;
            if (32 + col > lim) rb[col] = 0xff800000u;
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
      const float own = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      sm.xmax[w][j & 1][hh][row] = own;
      pair_sync(bar_id);
      const float mx = fmaxf(own, sm.xmax[w][j & 1][hh ^ 1][row]) * sc2;   // finite: key 128 j is visible
      const bool need = mx > m_used + kRescaleStep;      // also true on the first tile (m_used = -inf)
      if (j > 0 && __any_sync(0xffffffffu, need)) {
        // O of this tile must hold every PV issued so far before it is rescaled; both partner
        // warps hold the same rows and take this branch together
        ok = mbar_wait(&sm.o_done[w], (j - 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        const float f = need ? ex2(m_used - mx) : 1.f;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t o[32];
          tmem_ld32(my_o + ch * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int col = 0; col < 32; ++col) o[col] = __float_as_uint(__uint_as_float(o[col]) * f);
          tmem_st32(my_o + ch * 32, o);
        }
        l *= f;
      }
      if (need) m_used = mx;
      // pass 2: P = exp2(S * scale - m) over my 64 keys, written over S as bf16. P of keys
      // 64..127 lands on S columns 32..63, which the partner (keys 0..63) reads: it signals
      // once it holds them in registers, and the upper half waits for that before storing.
      float part[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t buf[2][32];
      tmem_ld32(my_s, buf[0]);
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t* cur = buf[ch];
        tmem_wait_ld();
        uint32_t zero = 0u;
        if (ch == 0) zero = tmem_ld32_zero(my_s + 32, buf[1]);   // in flight during this chunk's arithmetic
        if (ch == 1 && hh == 0) pair_arrive(bar_id);
        const float neg_m = __uint_as_float(zero) - m_used;
        if (diag) {
#pragma unroll
          for (int col = 0; col < 32; ++col)
            if (ch * 32 + col > lim) cur[col] = 0xff800000u;
        }
        uint32_t p[16];
#pragma unroll
        for (int c2 = 0; c2 < 16; ++c2) {
          const float p0 = ex2(fmaf(__uint_as_float(cur[2 * c2]), sc2, neg_m));
          const float p1 = ex2(fmaf(__uint_as_float(cur[2 * c2 + 1]), sc2, neg_m));
          part[c2 & 1] += p0;
          part[2 + (c2 & 1)] += p1;
          p[c2] = pack_bf16(p0, p1);
        }
        if (ch == 0 && hh == 1) pair_sync(bar_id);
        tmem_st16(my_p + ch * 16, p);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&sm.p_ready[w]);
      l += (part[0] + part[1]) + (part[2] + part[3]);
    }
    // row sum over both key halves, then my 64 columns of the output
    sm.xsum[w][hh][row] = l;
    pair_sync(bar_id);
    const float l_all = l + sm.xsum[w][hh ^ 1][row];
    if (ok && nkt_w > 0) ok = mbar_wait(&sm.o_done[w], (nkt_w - 1) & 1, abort_flag, a.status, code);
    if (ok && nkt_w > 0) {
      tc_fence_after();
      const float inv = 1.f / l_all;
      __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.out) + b * a.osb + h * a.osh + (int64_t)i * a.osn + hh * 64;
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t o[32];
        tmem_ld32(my_o + ch * 32, o);
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
      if (hh == 0 && i < n) a.lse[((int64_t)b * a.Hq + h) * n + i] = (m_used + log2f(l_all)) * kLn2;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kSoftmaxWarps) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

bool prefill_tc_supported(const PrefillArgs& a) {
  return a.dtype == PYR_BF16 && a.D == 128 && tensor_maps_available();
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
  attn_tc_kernel<<<grid, kThreads, smem, s>>>(mq, mk, mv, a);
  return cudaGetLastError();
}

}  // namespace pyr
