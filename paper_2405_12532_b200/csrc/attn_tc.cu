// tcgen05 causal attention of the prefill step (bf16, head_dim 128):
// Algorithm 1, "compute attention weights of KV", and the attention output.
//
// A CTA owns one (sequence, head) and walks its query rows in blocks of 256:
// two 128-row tiles that share every K and V tile the CTA loads (TMA, 128 keys
// per tile, two stages each). Because the CTA stays on the head, the loads, the
// first MMAs and the output epilogue of consecutive blocks overlap instead of
// paying a prologue per block, and every CTA of the grid does the same work.
//   warps 0-3 / 4-7   softmax of tile 0 / 1, thread = one query row
//   warp 8            MMA issue for both tiles (one lane)
//   warp 9            TMA loads (one lane)
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each. S covers 128 keys
// (one N = 128 MMA group, the shape that runs at full tensor rate); the softmax takes it as
// two halves of 64 keys, writes each half's P (bf16) over S columns 0..31 / 32..63 and
// signals it separately, so PV of the first half runs under the exponentials of the second.
// The issuing thread alternates between the tiles:
//     PVa0 PVb0 S0(j+1) | PVa1 PVb1 S1(j+1) | ...
// so one tile's softmax (bound by the ex2 unit) overlaps the other tile's tensor work.
// The running maximum used in the exponent is only raised when the row maximum has grown by
// more than 2^8, which keeps rescaling of O (a TMEM round trip) rare; the final normalisation
// uses the same maximum, so the result is the exact softmax.
//
// All mbarriers live across blocks, so every role counts the phases it has
// consumed (a parity wait is only valid one phase behind the barrier).
#include <cuda_bf16.h>

#include "pyr_internal.h"
#include "tc_common.cuh"

namespace pyr {
namespace {

using namespace tc;

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTile = 128;                  // query rows per tile, keys per K/V tile
constexpr int kHalf = 64;                   // keys per half-step
constexpr int kHalfBytes = kTile * 128;     // one [128 rows x 64 bf16] swizzled half tile (half of D)
constexpr int kTileBytes = 2 * kHalfBytes;  // a [128 x 128] bf16 tile = two halves along D
constexpr int kSoftmaxWarps = 8;
constexpr int kThreads = (kSoftmaxWarps + 2) * 32;
constexpr float kRescaleStep = 8.0f;

struct AttnSmem {
  alignas(1024) uint8_t q[2][kTileBytes];
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t v[2][kTileBytes];
  uint64_t q_full[2], q_empty[2];                    // per tile
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];   // per stage
  uint64_t s_full[2], pa_ready[2], pb_ready[2], o_done[2];   // per tile; P of keys 0..63 / 64..127
  uint32_t tmem_base;
  int abort_flag;
};

// Geometry of one 256-row block of the head.
struct Block {
  int r0, nkt0, nkt1, nkt;   // first row; key tiles of tile 0 / tile 1 (0 = tile absent) / loaded
};
__device__ __forceinline__ Block block_of(int blk, int n) {
  Block b;
  b.r0 = blk * 2 * kTile;
  b.nkt0 = 2 * blk + 1;                               // causal: the diagonal tile is the last one
  b.nkt1 = (b.r0 + kTile < n) ? 2 * blk + 2 : 0;
  b.nkt = b.nkt1 ? b.nkt1 : b.nkt0;
  return b;
}

// (10 warps put 3 on one scheduler partition: 16384 / (3 * 32) = 170 registers per thread at most)
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, PrefillArgs a) {
  extern __shared__ uint8_t smem_raw[];
  AttnSmem& sm = *reinterpret_cast<AttnSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int h = blockIdx.x, b = blockIdx.y;
  const int g = h / (a.Hq / a.Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = a.n;
  const int nblk = (n + 2 * kTile - 1) / (2 * kTile);
  volatile int* abort_flag = &sm.abort_flag;
  if (*reinterpret_cast<volatile int*>(a.status) != 0) return;   // an earlier CTA gave up: do not pile on

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.q_full[i], 1);
      mbar_init(&sm.q_empty[i], 1);
      mbar_init(&sm.k_full[i], 1);
      mbar_init(&sm.k_empty[i], 1);
      mbar_init(&sm.v_full[i], 1);
      mbar_init(&sm.v_empty[i], 1);
      mbar_init(&sm.o_done[i], 1);
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.pa_ready[i], kTile);
      mbar_init(&sm.pb_ready[i], kTile);
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
      bool ok = true;
      int kv = 0;                                      // K/V tiles loaded so far (stage = kv & 1)
      int nq[2] = {0, 0};                              // Q loads issued per tile
      for (int it = 0; it < nblk && ok; ++it) {
        const Block bk = block_of(nblk - 1 - it, n);   // longest block first
        for (int w = 0; w < 2 && ok; ++w) {
          if (w == 1 && !bk.nkt1) break;
          // the S MMAs of the previous block have finished reading this Q tile
          if (nq[w] > 0) ok = mbar_wait(&sm.q_empty[w], (nq[w] - 1) & 1, abort_flag, a.status, code);
          if (!ok) break;
          ++nq[w];
          mbar_expect_tx(&sm.q_full[w], kTileBytes);
          tma_load_4d(sm.q[w], &map_q, &sm.q_full[w], 0, h, bk.r0 + w * kTile, b);
          tma_load_4d(sm.q[w] + kHalfBytes, &map_q, &sm.q_full[w], 64, h, bk.r0 + w * kTile, b);
        }
        for (int j = 0; j < bk.nkt && ok; ++j, ++kv) {
          const int st = kv & 1;
          if (kv >= 2) ok = mbar_wait(&sm.k_empty[st], ((kv - 2) >> 1) & 1, abort_flag, a.status, code);
          if (!ok) break;
          mbar_expect_tx(&sm.k_full[st], kTileBytes);
          tma_load_4d(sm.k[st], &map_k, &sm.k_full[st], 0, g, j * kTile, b);
          tma_load_4d(sm.k[st] + kHalfBytes, &map_k, &sm.k_full[st], 64, g, j * kTile, b);
          if (kv >= 2) ok = mbar_wait(&sm.v_empty[st], ((kv - 2) >> 1) & 1, abort_flag, a.status, code);
          if (!ok) break;
          mbar_expect_tx(&sm.v_full[st], kTileBytes);
          tma_load_4d(sm.v[st], &map_v, &sm.v_full[st], 0, g, j * kTile, b);
          tma_load_4d(sm.v[st] + kHalfBytes, &map_v, &sm.v_full[st], 64, g, j * kTile, b);
        }
      }
    }
    __syncwarp();
  } else if (warp == kSoftmaxWarps) {
    // ---------------------------------------------------------------- MMA issue (one thread, both tiles)
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(kTile, kTile, false, false);   // S = Q K^T, both K-major
      constexpr uint32_t idesc_o = idesc_bf16(kTile, kTile, false, true);    // O += P V, V is MN-major
      // operand descriptors are built once; a k-step only adds a constant to the start-address field
      const uint64_t dq0 = smem_desc_sw128(smem_u32(sm.q[0]), 16, 1024), dq1 = smem_desc_sw128(smem_u32(sm.q[1]), 16, 1024);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, 1024), dk1 = smem_desc_sw128(smem_u32(sm.k[1]), 16, 1024);
      const uint64_t dv0 = smem_desc_sw128(smem_u32(sm.v[0]), kHalfBytes, 1024);
      const uint64_t dv1 = smem_desc_sw128(smem_u32(sm.v[1]), kHalfBytes, 1024);
      bool ok = true;
      int kvu = 0;             // K/V tiles of the ring that earlier blocks used
      int nq[2] = {0, 0};      // Q loads consumed per tile
      int cnt[2] = {0, 0};     // key tiles done per tile in earlier blocks
      for (int it = 0; it < nblk && ok; ++it) {
        const Block bk = block_of(nblk - 1 - it, n);
        const int last_w = bk.nkt1 ? 1 : 0;
        auto issue_s = [&](int w, int j, int st) {
          const uint64_t qd = w ? dq1 : dq0, kd = st ? dk1 : dk0;
          const uint32_t d_tmem = tmem + w * kTile;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
            mma_ss(d_tmem, qd + off, kd + off, idesc_s, kk > 0);
          }
          mma_commit(&sm.s_full[w]);
          if (j == (w ? bk.nkt1 : bk.nkt0) - 1) mma_commit(&sm.q_empty[w]);   // last read of this block's Q tile
        };
        // PV over 64 keys: half 0 = P columns 0..31 and V rows 0..63, half 1 = the rest
        auto issue_pv = [&](int w, int st, int half, bool accumulate) {
          const uint64_t vd = (st ? dv1 : dv0) + (uint64_t)((half * kHalf * 128) >> 4);
          const uint32_t d_tmem = tmem + (2 + w) * kTile, p_tmem = tmem + w * kTile + half * 32;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)   // 16 keys per step: 8 TMEM columns of P, 16 rows of V
            mma_ts(d_tmem, p_tmem + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), idesc_o, (accumulate || kk > 0) ? 1u : 0u);
          mma_commit(&sm.o_done[w]);
        };
        for (int w = 0; w <= last_w && ok; ++w) {
          ok = mbar_wait(&sm.q_full[w], nq[w] & 1, abort_flag, a.status, code);
          ++nq[w];
        }
        if (ok) ok = mbar_wait(&sm.k_full[kvu & 1], (kvu >> 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        issue_s(0, 0, kvu & 1);
        if (last_w) issue_s(1, 0, kvu & 1);
        mma_commit(&sm.k_empty[kvu & 1]);
        // Order per key tile j: PVa0 PVb0 S0(j+1) PVa1 PVb1 S1(j+1). While one tile's softmax runs,
        // the other tile's groups keep the tensor pipe busy.
        for (int j = 0; j < bk.nkt && ok; ++j) {
          const int ring = kvu + j, st = ring & 1, st1 = (ring + 1) & 1;
          ok = mbar_wait(&sm.v_full[st], (ring >> 1) & 1, abort_flag, a.status, code);
          if (!ok) break;
          bool k_next_ready = false;
          for (int w = 0; w < 2 && ok; ++w) {
            const int nkt_w = w ? bk.nkt1 : bk.nkt0;
            if (j < nkt_w) {
              const int par = (cnt[w] + j) & 1;
              ok = mbar_wait(&sm.pa_ready[w], par, abort_flag, a.status, code);
              if (!ok) break;
              tc_fence_after();
              issue_pv(w, st, 0, j > 0);
              ok = mbar_wait(&sm.pb_ready[w], par, abort_flag, a.status, code);
              if (!ok) break;
              tc_fence_after();
              issue_pv(w, st, 1, true);
            }
            if (w == last_w) mma_commit(&sm.v_empty[st]);
            if (j + 1 < nkt_w) {
              if (!k_next_ready) {
                ok = mbar_wait(&sm.k_full[st1], ((ring + 1) >> 1) & 1, abort_flag, a.status, code);
                if (!ok) break;
                k_next_ready = true;
                tc_fence_after();
              }
              issue_s(w, j + 1, st1);
            }
            if (w == last_w && j + 1 < bk.nkt) mma_commit(&sm.k_empty[st1]);
          }
        }
        kvu += bk.nkt;
        cnt[0] += bk.nkt0;
        cnt[1] += bk.nkt1;
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- softmax, thread = query row
    const int w = warp >> 2;
    const int row = threadIdx.x & (kTile - 1);
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_addr = tmem + lane_base + w * kTile;          // S (128 columns); P lands on columns 0..63
    const uint32_t o_addr = tmem + lane_base + (2 + w) * kTile;
    const float sc2 = a.scale * kLog2e;
    bool ok = true;
    int cnt = 0;    // key tiles of this tile done in earlier blocks
    for (int it = 0; it < nblk && ok; ++it) {
      const Block bk = block_of(nblk - 1 - it, n);
      const int nkt_w = w ? bk.nkt1 : bk.nkt0;
      if (nkt_w == 0) continue;
      const int i = bk.r0 + w * kTile + row;             // query row of this thread
      float m_used = -INFINITY, l = 0.f;
      // one online-softmax step over 64 keys held in s[0..63]; P goes to 32 columns at p_addr.
      // `od` = index of the o_done phase that must be complete before O may be rescaled.
      auto half_step = [&](uint32_t* s, int lim, bool diag, bool first, uint32_t p_addr, int od, uint64_t* ready) {
        if (diag) {
#pragma unroll
          for (int col = 0; col < 64; ++col)
            if (col > lim) s[col] = 0xff800000u;   // -inf: key not visible to this row
        }
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int col = 0; col < 64; col += 8) {
          mx0 = max3(mx0, __uint_as_float(s[col]), __uint_as_float(s[col + 1]));
          mx1 = max3(mx1, __uint_as_float(s[col + 2]), __uint_as_float(s[col + 3]));
          mx2 = max3(mx2, __uint_as_float(s[col + 4]), __uint_as_float(s[col + 5]));
          mx3 = max3(mx3, __uint_as_float(s[col + 6]), __uint_as_float(s[col + 7]));
        }
        // (-inf when every key of this half is hidden from the row: then nothing changes and P = 0)
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sc2;
        const bool need = mx > m_used + kRescaleStep;      // also true on the first half (m_used = -inf)
        bool followed = false;
        if (!first && __any_sync(0xffffffffu, need)) {
          // O must hold every PV issued so far before it is rescaled
          ok = mbar_wait(&sm.o_done[w], od & 1, abort_flag, a.status, code);
          followed = true;
          if (!ok) return;
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
        const float neg_m = -m_used;
        float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t p[16];
#pragma unroll
          for (int c2 = 0; c2 < 16; ++c2) {
            const float p0 = ex2(fmaf(__uint_as_float(s[ch * 32 + 2 * c2]), sc2, neg_m));
            const float p1 = ex2(fmaf(__uint_as_float(s[ch * 32 + 2 * c2 + 1]), sc2, neg_m));
            part[c2 & 1] += p0;
            part[2 + (c2 & 1)] += p1;
            p[c2] = pack_bf16(p0, p1);
          }
          tmem_st16(p_addr + ch * 16, p);
        }
        l += (part[0] + part[1]) + (part[2] + part[3]);
        // a parity wait is only valid one phase behind the barrier: follow o_done on every half
        // (by now the PV in question was issued a whole half-step ago, so this is normally free)
        if (!first && !followed) ok = mbar_wait(&sm.o_done[w], od & 1, abort_flag, a.status, code);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(ready);
      };
      for (int j = 0; j < nkt_w && ok; ++j) {
        ok = mbar_wait(&sm.s_full[w], (cnt + j) & 1, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        uint32_t sa[64], sb[64];
        tmem_ld32(s_addr, sa);
        tmem_ld32(s_addr + 32, sa + 32);
        tmem_ld32(s_addr + 64, sb);
        tmem_ld32(s_addr + 96, sb + 32);
        tmem_wait_ld();
        const bool diag = j == nkt_w - 1;          // key 128 j + col is visible iff col <= i - 128 j
        const int lim = i - j * kTile;
        const int od = 2 * (cnt + j);              // o_done phases: 2 j = PVa(j), 2 j + 1 = PVb(j)
        half_step(sa, lim, diag, j == 0, s_addr, od - 1, &sm.pa_ready[w]);
        if (!ok) break;
        half_step(sb, lim - kHalf, diag, false, s_addr + 32, od, &sm.pb_ready[w]);
      }
      // epilogue of the block; the next block's first PV cannot start before these threads have
      // delivered its P, i.e. after they are done reading O here
      if (ok) ok = mbar_wait(&sm.o_done[w], (2 * (cnt + nkt_w) - 1) & 1, abort_flag, a.status, code);
      if (!ok) break;
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
      if (i < n) a.lse[((int64_t)b * a.Hq + h) * n + i] = (m_used + log2f(l)) * kLn2;
      cnt += nkt_w;
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
  dim3 grid(a.Hq, a.B);
  attn_tc_kernel<<<grid, kThreads, smem, s>>>(mq, mk, mv, a);
  return cudaGetLastError();
}

}  // namespace pyr
