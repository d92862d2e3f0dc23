// tcgen05 causal attention of the prefill step (bf16, head_dim 128):
// Algorithm 1, "compute attention weights of KV", and the attention output.
//
// A CTA owns one (sequence, head), or one of 2, 4 or 8 shares of it when there
// are too few heads to fill the SMs evenly, and walks its 128-row query tiles
// one at a time, longest first (key tiles up in even tiles of the walk and down
// in odd ones, so that a tile starts on K/V still in L2). The K tiles of all
// query tiles form one stream r = 0, 1, 2, ... that every role walks on its own.
//   warps 0-3   softmax group 0, thread = one query row
//   warps 4-7   softmax group 1 (same rows), and the epilogue of every tile
//   warp 8      issues the S MMAs:  S(r) = Q K(r)^T, 128 keys, Q and K from shared memory
//   warp 9      TMA loads of Q and K (two stages of K)
//   warp 10     issues the PV MMAs: O += P(r) V(r), P from tensor memory
//   warp 11     TMA loads of V (two stages; a V stage is freed up to three K tiles after the
//               K stage, so the K loads must not queue behind the V loads)
// Tensor memory (512 columns): three S buffers of 128 fp32 columns (K tile r uses
// buffer r % 3; P as bf16 overwrites the first 64 columns) and O (128 columns).
// S(r) may be issued as soon as PV(r - 3) has read its P, so the S MMAs run up to
// three K tiles ahead of the softmax and never wait for it; separate issuing
// threads keep either kind of MMA from queueing behind the other's waits.
// Within a query tile the two softmax groups take alternate K tiles, counted
// from the tile's end, so group 1 always has the last one and writes the tile
// out. A thread holds its row's 128 scores in registers (the four issuing and
// loading warps hand their registers to the softmax warps at the start). What
// couples the groups is the maximum used in the exponent: the thread of K tile
// r reads the value published for r - 1, raises it only when the row maximum
// has grown by more than 2^8 (which keeps rescaling of O, a TMEM round trip,
// rare), and publishes its own before it starts on the exponentials. Each group
// keeps its own row sum; the epilogue adds them under the final maximum, so
// the result is the exact softmax.
//
// All mbarriers live across tiles, so every role counts the phases it has
// consumed (a parity wait is only valid one phase behind the barrier; the
// waits that do not follow a barrier phase by phase say why they still are).
#include <cuda_bf16.h>
#include <stddef.h>

#include "pyr_internal.h"
#include "tc_common.cuh"

namespace pyr {
namespace {

using namespace tc;

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTile = 128;                  // query rows per tile, keys per K/V tile
constexpr int kHalfBytes = kTile * 128;     // one [128 rows x 64 bf16] swizzled half tile (half of D)
constexpr int kTileBytes = 2 * kHalfBytes;  // a [128 x 128] bf16 tile = two halves along D
constexpr int kSoftmaxWarps = 8;
constexpr int kThreads = (kSoftmaxWarps + 4) * 32;
constexpr float kRescaleStep = 8.0f;
constexpr int kRegsLaunch = 168, kRegsSoftmax = 232, kRegsIssue = 40;   // kRegsLaunch must be what ptxas reports for the kernel
constexpr int kSBufs = 3;                   // S buffers of 128 fp32 columns: TMEM columns 0..383
constexpr uint32_t kColO = 384;             // O: columns 384..511

struct AttnSmem {
  alignas(1024) uint8_t q[2][kTileBytes];
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t v[2][kTileBytes];
  alignas(1024) uint8_t o_stage[kTileBytes];         // a [128 x 128] bf16 tile of O on its way out
  unsigned long long m_slot[kTile];                  // per row: (K tiles decided so far) << 32 | bits of the maximum in use
  float l_even[2][kTile];                            // [tile parity][row]: group 0's row sum of the tile
  uint64_t q_full[2], q_empty[2];                    // per Q buffer
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];   // per stage
  uint64_t s_full[3], p_ready[3], pv_done[3];        // per S buffer (K tile r of the stream uses buffer r % 3): S landed / P written / PV has read P
  uint64_t o_free;                                   // the epilogue has read O
  uint32_t tmem_base;
  int abort_flag;
};
// bytes in use (the struct's size is rounded up to its 1024-byte alignment)
constexpr size_t kSmemNeed = offsetof(AttnSmem, abort_flag) + sizeof(int);

// One tile of the walk.
struct Tile {
  int r0, nkt;   // first row; key tiles (causal: the diagonal tile is the last one)
};

// A head's tiles can be dealt to `parts` CTAs. With the tiles numbered from the longest (k = 0),
// part p takes k = p, 2 parts - 1 - p, 2 parts + p, 4 parts - 1 - p, ...: a long tile is paired with
// a short one, so the parts carry nearly equal work. Returns false when the part has no it-th tile.
__host__ __device__ __forceinline__ bool tile_at(int it, int part, int parts, int n, Tile* tl) {
  const int ntiles = (n + kTile - 1) / kTile;
  const int k = 2 * parts * (it >> 1) + ((it & 1) ? 2 * parts - 1 - part : part);
  if (k >= ntiles) return false;
  const int ti = ntiles - 1 - k;
  tl->r0 = ti * kTile;
  tl->nkt = ti + 1;
  return true;
}

__device__ __forceinline__ bool slot_wait(const volatile unsigned long long* slot, uint32_t seq, float* m,
                                          volatile int* abort_flag, int* status, int code) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    const unsigned long long x = *slot;
    if ((uint32_t)(x >> 32) == seq) {
      *m = __uint_as_float((uint32_t)x);
      return true;
    }
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  if (status) atomicCAS(status, 0, code);
  return false;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                PrefillArgs a, int parts) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // The tiles need 1024-byte alignment. The launch asks for what the struct needs plus as much of
  // a kilobyte as the SM's limit leaves; if the window's base is not aligned well enough for that,
  // the CTA reports it instead of running past the end.
  const uint32_t pad = (1024u - (smem_u32(smem_raw) & 1023u)) & 1023u;
  uint32_t dyn_bytes;
  asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_bytes));
  if (pad + kSmemNeed > dyn_bytes) {
    if (threadIdx.x == 0) atomicCAS(a.status, 0, (int)PYR_ERR_CUDA);
    return;
  }
  AttnSmem& sm = *reinterpret_cast<AttnSmem*>(smem_raw + pad);

  const int h = blockIdx.x / parts, part = blockIdx.x % parts, b = blockIdx.y;
  const int g = h / (a.Hq / a.Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = a.n;
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
    }
    for (int i = 0; i < kSBufs; ++i) {
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.p_ready[i], kTile);
      mbar_init(&sm.pv_done[i], 1);
    }
    mbar_init(&sm.o_free, kTile);
    sm.abort_flag = 0;
    fence_barrier_init();
  }
  if (threadIdx.x < kTile) sm.m_slot[threadIdx.x] = 0ull;
  if (warp == kSoftmaxWarps) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const int code = PYR_ERR_TIMEOUT;
  // Register split: the block starts with kThreads x kRegsLaunch registers; the four issuing /
  // loading warps (one warpgroup) give theirs up, the two softmax warpgroups take them:
  // 256 x kRegsSoftmax + 128 x kRegsIssue <= kThreads x kRegsLaunch.
  static_assert(256 * kRegsSoftmax + 128 * kRegsIssue <= kThreads * kRegsLaunch, "register split exceeds the launch's total");

  if (warp >= kSoftmaxWarps) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssue));
  if (warp == kSoftmaxWarps + 1) {
    // ---------------------------------------------------------------- TMA loads of Q and K
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      bool ok = true;
      int kv = 0;                                      // K/V tiles loaded so far (stage = kv & 1)
      // Q of tile `it` goes into buffer it & 1 once the S MMAs of tile it - 2 have read it.
      auto load_q = [&](int it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, &tl)) return;
        const int bq = it & 1;
        if (it >= 2) ok = mbar_wait(&sm.q_empty[bq], ((it - 2) >> 1) & 1, abort_flag, a.status, code);
        if (!ok) return;
        mbar_expect_tx(&sm.q_full[bq], kTileBytes);
        tma_load_4d(sm.q[bq], &map_q, &sm.q_full[bq], 0, h, tl.r0, b);
        tma_load_4d(sm.q[bq] + kHalfBytes, &map_q, &sm.q_full[bq], 64, h, tl.r0, b);
      };
      load_q(0);
      for (int it = 0; ok; ++it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, &tl)) break;   // longest tile first
        // Key tiles go up in even tiles of the walk and down in odd ones: the tiles read last are
        // the first ones the next tile reads, so they are still in L2.
        const bool down = it & 1;
        for (int jj = 0; jj < tl.nkt && ok; ++jj, ++kv) {
          const int j = down ? tl.nkt - 1 - jj : jj;
          const int st = kv & 1;
          if (kv >= 2) ok = mbar_wait(&sm.k_empty[st], ((kv - 2) >> 1) & 1, abort_flag, a.status, code);
          if (!ok) break;
          mbar_expect_tx(&sm.k_full[st], kTileBytes);
          tma_load_4d(sm.k[st], &map_k, &sm.k_full[st], 0, g, j * kTile, b);
          tma_load_4d(sm.k[st] + kHalfBytes, &map_k, &sm.k_full[st], 64, g, j * kTile, b);
          // The next tile's Q follows this tile's first K/V tile: early enough for the S MMAs, which
          // run ahead into the next tile, and late enough not to hold up that K/V tile while the
          // tile before is still reading the Q buffer.
          if (jj == 0) load_q(it + 1);
        }
      }
    }
    __syncwarp();
  } else if (warp == kSoftmaxWarps + 3) {
    // ---------------------------------------------------------------- TMA loads of V
    // (a thread of their own: a V stage is released by its PV, up to three K tiles after the S
    // MMAs released the K stage, and the K loads must not wait for that)
    if (lane == 0) {
      prefetch_tensormap(&map_v);
      bool ok = true;
      int kv = 0;
      for (int it = 0; ok; ++it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, &tl)) break;
        const bool down = it & 1;
        for (int jj = 0; jj < tl.nkt && ok; ++jj, ++kv) {
          const int j = down ? tl.nkt - 1 - jj : jj;
          const int st = kv & 1;
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
    // ---------------------------------------------------------------- S MMAs: S(r) = Q K^T for K tile r of the stream
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(kTile, kTile, false, false);   // both K-major
      const uint64_t dq0 = smem_desc_sw128(smem_u32(sm.q[0]), 16, 1024), dq1 = smem_desc_sw128(smem_u32(sm.q[1]), 16, 1024);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, 1024), dk1 = smem_desc_sw128(smem_u32(sm.k[1]), 16, 1024);
      bool ok = true;
      int ring = 0, sb = 0, sph = 0;                   // K tiles so far; S buffer ring % 3 and the parity of ring / 3
      for (int it = 0; ok; ++it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, &tl)) break;
        const int bq = it & 1;
        ok = mbar_wait(&sm.q_full[bq], (it >> 1) & 1, abort_flag, a.status, code);
        const uint64_t dq = bq ? dq1 : dq0;
        for (int j = 0; j < tl.nkt && ok; ++j, ++ring) {
          const int st = ring & 1;
          ok = mbar_wait(&sm.k_full[st], (ring >> 1) & 1, abort_flag, a.status, code);
          // the buffer is free once PV(ring - 3) has read its P
          if (ok && ring >= kSBufs) ok = mbar_wait(&sm.pv_done[sb], sph ^ 1, abort_flag, a.status, code);
          if (!ok) break;
          tc_fence_after();
          const uint64_t kd = st ? dk1 : dk0;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
            mma_ss(tmem + sb * kTile, dq + off, kd + off, idesc_s, kk > 0);
          }
          mma_commit(&sm.s_full[sb]);
          mma_commit(&sm.k_empty[st]);
          if (j == tl.nkt - 1) mma_commit(&sm.q_empty[bq]);     // last read of this Q tile
          if (++sb == kSBufs) { sb = 0; sph ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == kSoftmaxWarps + 2) {
    // ---------------------------------------------------------------- PV MMAs: O += P(r) V
    if (lane == 0) {
      constexpr uint32_t idesc_o = idesc_bf16(kTile, kTile, false, true);    // V is MN-major
      const uint64_t dv0 = smem_desc_sw128(smem_u32(sm.v[0]), kHalfBytes, 1024);
      const uint64_t dv1 = smem_desc_sw128(smem_u32(sm.v[1]), kHalfBytes, 1024);
      const uint32_t o_tmem = tmem + kColO;
      bool ok = true;
      int ring = 0, sb = 0, sph = 0;
      for (int it = 0; ok; ++it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, &tl)) break;
        // the first PV of a tile overwrites the accumulator of the tile before it
        if (it >= 1) ok = mbar_wait(&sm.o_free, (it - 1) & 1, abort_flag, a.status, code);
        for (int j = 0; j < tl.nkt && ok; ++j, ++ring) {
          const int st = ring & 1;
          ok = mbar_wait(&sm.v_full[st], (ring >> 1) & 1, abort_flag, a.status, code);
          if (ok) ok = mbar_wait(&sm.p_ready[sb], sph, abort_flag, a.status, code);
          if (!ok) break;
          tc_fence_after();
          const uint64_t vd = st ? dv1 : dv0;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)   // 16 keys per MMA: 8 TMEM columns of P, 16 rows of V
            mma_ts(o_tmem, tmem + sb * kTile + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), idesc_o,
                   (j > 0 || kk > 0) ? 1u : 0u);
          mma_commit(&sm.pv_done[sb]);
          mma_commit(&sm.v_empty[st]);
          if (++sb == kSBufs) { sb = 0; sph ^= 1; }
        }
      }
    }
    __syncwarp();
  }
  } else {
    // ---------------------------------------------------------------- softmax, thread = query row
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    const int grp = warp >> 2;                           // 1: takes every tile's last K tile, and the epilogue
    const int row = threadIdx.x & (kTile - 1);
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_base = tmem + lane_base;
    const uint32_t o_addr = t_base + kColO;
    const float sc2 = a.scale * kLog2e;
    bool ok = true;
    int ring0 = 0;               // K tiles of earlier tiles

    for (int it = 0; ok; ++it) {
      Tile tl;
      if (!tile_at(it, part, parts, n, &tl)) break;
      const int nkt = tl.nkt;
      const int i = tl.r0 + row;                          // query row of this thread
      const int tp = it & 1;
      float m_mine = -INFINITY, l = 0.f;                  // this group's row sum and the maximum it is relative to
      float m_other = -INFINITY;                          // (group 1) the maximum group 0's row sum is relative to
      // The groups alternate within the tile, counted from its end: group 1 has the last K tile.
      for (int j = (((nkt - 1) & 1) == grp) ? 1 : 0; j < nkt && ok; j += 2) {
        const int ring = ring0 + j;
        const int sb = ring % kSBufs, sph = (ring / kSBufs) & 1;
        const uint32_t s_addr = t_base + sb * kTile;
        ok = mbar_wait(&sm.s_full[sb], sph, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        // key tile of this step: ascending in even tiles of the walk, descending in odd ones
        const int kt = (it & 1) ? nkt - 1 - j : j;
        const bool diag = kt == nkt - 1;    // inside the diagonal key tile key 128 kt + col is visible iff col <= i - 128 kt
        const int lim = i - kt * kTile;
        uint32_t s[kTile];               // the row's 128 scores (the softmax warps hold the registers for it)
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) tmem_ld32(s_addr + ch * 32, s + ch * 32);
        tmem_wait_ld();
        if (diag) {
#pragma unroll
          for (int col = 0; col < kTile; ++col)
            if (col > lim) s[col] = 0xff800000u;   // -inf
        }
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int col = 0; col < kTile; col += 8) {
          mx0 = max3(mx0, __uint_as_float(s[col]), __uint_as_float(s[col + 1]));
          mx1 = max3(mx1, __uint_as_float(s[col + 2]), __uint_as_float(s[col + 3]));
          mx2 = max3(mx2, __uint_as_float(s[col + 4]), __uint_as_float(s[col + 5]));
          mx3 = max3(mx3, __uint_as_float(s[col + 6]), __uint_as_float(s[col + 7]));
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sc2;   // finite: column 0 of the tile is visible
        // The maximum in use after the K tile before this one, from the thread that took it (the
        // partner of this row, or this thread itself across a tile border). A tile's first K tile
        // starts from -inf but still waits: the slot is one word per row.
        float m_prev = -INFINITY;
        if (ring > 0) ok = slot_wait(&sm.m_slot[row], (uint32_t)ring, &m_prev, abort_flag, a.status, code);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (j == 0) m_prev = -INFINITY;
        m_other = m_prev;
        const bool need = mx > m_prev + kRescaleStep;      // always true on the first K tile of a tile
        const float m_used = need ? mx : m_prev;
        *reinterpret_cast<volatile unsigned long long*>(&sm.m_slot[row]) =
            ((unsigned long long)(uint32_t)(ring + 1) << 32) | __float_as_uint(m_used);
        if (j > 0 && __any_sync(0xffffffffu, need)) {
          // O may be rescaled once PV(ring - 1) is complete. (That barrier's phases are not followed
          // one by one here, but it is exactly at this one: PV(ring - 4) had to be complete before
          // S(ring - 1) was issued, and PV(ring + 2) comes after PV(ring), which needs the P this
          // thread has yet to write.)
          ok = mbar_wait(&sm.pv_done[(ring - 1) % kSBufs], ((ring - 1) / kSBufs) & 1, abort_flag, a.status, code);
          if (!ok) break;
          tc_fence_after();
          const float f = need ? ex2(m_prev - m_used) : 1.f;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t o[32];
            tmem_ld32(o_addr + ch * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int col = 0; col < 32; ++col) o[col] = __float_as_uint(__uint_as_float(o[col]) * f);
            tmem_st32(o_addr + ch * 32, o);
          }
        }
        if (m_used != m_mine) {          // bring this group's row sum under the maximum now in use
          l *= ex2(m_mine - m_used);
          m_mine = m_used;
        }
        const float neg_m = -m_used;
        float part4[4] = {0.f, 0.f, 0.f, 0.f};
        // P = exp2(S - m) as bf16 overwrites the first 64 columns of the buffer (S is in registers)
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t p[16];
#pragma unroll
          for (int c2 = 0; c2 < 16; ++c2) {
            const float p0 = ex2(fmaf(__uint_as_float(s[ch * 32 + 2 * c2]), sc2, neg_m));
            const float p1 = ex2(fmaf(__uint_as_float(s[ch * 32 + 2 * c2 + 1]), sc2, neg_m));
            part4[c2 & 1] += p0;
            part4[2 + (c2 & 1)] += p1;
            p[c2] = pack_bf16(p0, p1);
          }
          tmem_st16(s_addr + ch * 16, p);
        }
        l += (part4[0] + part4[1]) + (part4[2] + part4[3]);
        // Group 0's row sum of the tile (relative to the maximum after K tile nkt - 2, which group 1
        // reads for the last K tile) goes to the epilogue before the arrival for P(nkt - 2): the
        // epilogue runs after PV(nkt - 1), which is issued after PV(nkt - 2), which follows that arrival.
        if (grp == 0 && j == nkt - 2) sm.l_even[tp][row] = l;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&sm.p_ready[sb]);
      }
      if (grp == 1) {
        // Epilogue of the tile (group 1 took the last K tile, so m_mine is the final maximum). A
        // thread whose wait ran out still goes to the barrier, and the barrier itself tells all
        // 128 threads whether any of them did.
        const int rl = ring0 + nkt - 1;
        if (ok) ok = mbar_wait(&sm.pv_done[rl % kSBufs], (rl / kSBufs) & 1, abort_flag, a.status, code);
        if (row == 0) bulk_wait_read_all();      // the stores of the tile before have read the staging tile
        uint32_t any_bad;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, 128, q;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(any_bad)
            : "r"((uint32_t)(ok ? 0 : 1))
            : "memory");
        if (any_bad) { ok = false; break; }
        tc_fence_after();
        if (nkt >= 2) l += *reinterpret_cast<volatile float*>(&sm.l_even[tp][row]) * ex2(m_other - m_mine);
        if (i < n) a.lse[((int64_t)b * a.Hq + h) * n + i] = (m_mine + log2f(l)) * kLn2;
        const float inv = 1.f / l;
        // O leaves through shared memory and two TMA stores (rows past n are clipped by the store)
        uint8_t* my_row = sm.o_stage + row * 128;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t o[64];
          tmem_ld32(o_addr + hf * 64, o);
          tmem_ld32(o_addr + hf * 64 + 32, o + 32);
          tmem_wait_ld();
          if (hf == 1) {           // the accumulator is in registers: the next tile may overwrite it
            tc_fence_before();
            mbar_arrive(&sm.o_free);
          }
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {     // 16-byte chunk ch of the row sits at ch ^ (row & 7): the 128-byte swizzle
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(o[ch * 8 + 0]) * inv, __uint_as_float(o[ch * 8 + 1]) * inv);
            pk.y = pack_bf16(__uint_as_float(o[ch * 8 + 2]) * inv, __uint_as_float(o[ch * 8 + 3]) * inv);
            pk.z = pack_bf16(__uint_as_float(o[ch * 8 + 4]) * inv, __uint_as_float(o[ch * 8 + 5]) * inv);
            pk.w = pack_bf16(__uint_as_float(o[ch * 8 + 6]) * inv, __uint_as_float(o[ch * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(my_row + hf * kHalfBytes + ((ch ^ (row & 7)) << 4)) = pk;
          }
        }
        fence_proxy_async();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (row == 0) {
          tma_store_4d(&map_o, sm.o_stage, 0, h, tl.r0, b);
          tma_store_4d(&map_o, sm.o_stage + kHalfBytes, 64, h, tl.r0, b);
          bulk_commit();
        }
      }
      if (!ok) break;
      ring0 += nkt;
    }
    if (grp == 1 && row == 0) bulk_wait_all();   // the last stores have left shared memory and are complete
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
  CUtensorMap mq, mk, mv, mo;
  if (!make_tensor_map_bf16(&mo, a.out, a.B, a.n, a.Hq, a.D, a.osb, a.osn, a.osh, kTile) ||
      !make_tensor_map_bf16(&mq, a.q, a.B, a.n, a.Hq, a.D, a.qsb, a.qsn, a.qsh, kTile) ||
      !make_tensor_map_bf16(&mk, a.k, a.B, a.n, a.Hkv, a.D, a.ksb, a.ksn, a.ksh, kTile) ||
      !make_tensor_map_bf16(&mv, a.v, a.B, a.n, a.Hkv, a.D, a.ksb, a.ksn, a.ksh, kTile))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0, smem_max = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
  // the register split inside the kernel is sized for kRegsLaunch registers per thread at launch
  cudaFuncAttributes fa;
  if ((e = cudaFuncGetAttributes(&fa, attn_tc_kernel)) != cudaSuccess) return e;
  if (fa.numRegs != kRegsLaunch) return cudaErrorInvalidConfiguration;
  size_t smem = kSmemNeed + 1024;
  if (smem > (size_t)smem_max) smem = (size_t)smem_max;
  if (smem < kSmemNeed) return cudaErrorInvalidConfiguration;
  e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // One CTA per (sequence, head) when that fills the SMs evenly; otherwise deal each head's tiles
  // to 2, 4 or 8 CTAs. Cost model: waves of CTAs x the largest share of key-tile steps a CTA gets
  // (a tile costs about one step more, a CTA about two); splitting must win by 5 % to be chosen.
  const int ntiles = (a.n + kTile - 1) / kTile;
  const long long heads = (long long)a.Hq * a.B;
  int parts = 1;
  long long best = -1;
  for (int p = 1; p <= 8 && p <= ntiles; p *= 2) {
    long long share = 0;                       // key-tile steps of the busiest part
    for (int part = 0; part < p; ++part) {
      long long w = 0;
      Tile tl;
      for (int it = 0; tile_at(it, part, p, a.n, &tl); ++it) w += tl.nkt + 1;
      if (w + 2 > share) share = w + 2;
    }
    const long long cost = ((heads * p + sms - 1) / sms) * share;
    if (best < 0 || cost * 100 < best * 95) { best = cost; parts = p; }
  }
  dim3 grid(a.Hq * parts, a.B);
  attn_tc_kernel<<<grid, kThreads, smem, s>>>(mq, mk, mv, mo, a, parts);
  return cudaGetLastError();
}

}  // namespace pyr
