// tcgen05 causal attention of the prefill step (bf16, head_dim 128):
// Algorithm 1, "compute attention weights of KV", and the attention output.
//
// A CTA owns one (sequence, head), or one of 2, 4 or 8 equal shares of it when
// there are too few heads to fill the SMs evenly, and walks its query rows in
// blocks of 256: two 128-row tiles that share every K and V tile the CTA loads
// (TMA, 128 keys per tile, two stages each; up through the key tiles in even
// blocks and down in odd ones, so that a block starts on tiles still in L2).
// Because the CTA stays on the head, the loads, the first MMAs and the output
// epilogue (a staged tile and two TMA stores) of consecutive blocks overlap
// instead of paying a prologue per block, and every CTA does the same work.
//   warps 0-3 / 4-7   softmax of tile 0 / 1, thread = one query row
//   warp 8 / 9        MMA issue for tile 0 / 1 (one lane each)
//   warp 10           TMA loads (one lane)
// The keys are consumed in half-steps of 64. Tensor memory, per tile 256 of the
// 512 columns: two S buffers of 64 fp32 columns and O (128 columns); P (bf16)
// overwrites the first 32 columns of its S buffer. Because S is double
// buffered, the issuing thread runs S(t+1) while the softmax of half-step t is
// at work, and PV(t) follows as soon as P(t) is there:
//     S(0) S(1) | PV(0) S(2) | PV(1) S(3) | ...
// The running maximum used in the exponent is only raised when the row maximum
// has grown by more than 2^8, which keeps rescaling of O (a TMEM round trip)
// rare; the final normalisation uses the same maximum, so the result is the
// exact softmax.
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
constexpr int kThreads = (kSoftmaxWarps + 3) * 32;
constexpr float kRescaleStep = 8.0f;

struct AttnSmem {
  alignas(1024) uint8_t q[2][kTileBytes];
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t v[2][kTileBytes];
  alignas(1024) uint8_t o_stage[kTileBytes];         // a [128 x 128] bf16 tile of O on its way out (both tiles use it)
  uint64_t q_full[2], q_empty[2];                    // per tile
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];   // per stage; empty = both issuing threads arrived
  uint64_t s_full[2][2], p_ready[2][2], o_done[2][2];   // [tile][S buffer]
  uint64_t stage_free;                               // the stores of one epilogue have read o_stage
  uint32_t tmem_base;
  int abort_flag;
};

// Geometry of one block of the head: two consecutive 128-row tiles that share their K/V tiles.
// The tiles are paired from the last one down, so that with an odd number of tiles the block that
// has a single tile is the one with the least work (the first 128 rows), not the one with the most.
struct Block {
  int r0, nkt0, nkt1, nkt;   // first row; key tiles of tile 0 / tile 1 (0 = tile absent) / loaded
};
__host__ __device__ __forceinline__ Block block_of(int blk, int n) {
  const int ntiles = (n + kTile - 1) / kTile;
  Block b;
  if (ntiles & 1) {
    b.r0 = blk ? (2 * blk - 1) * kTile : 0;
    b.nkt0 = blk ? 2 * blk : 1;                         // causal: the diagonal tile is the last one
    b.nkt1 = blk ? 2 * blk + 1 : 0;
  } else {
    b.r0 = blk * 2 * kTile;
    b.nkt0 = 2 * blk + 1;
    b.nkt1 = 2 * blk + 2;
  }
  b.nkt = b.nkt1 ? b.nkt1 : b.nkt0;
  return b;
}

// A head's blocks can be dealt to `parts` CTAs (used when there are too few heads to fill the SMs
// evenly). With the blocks numbered from the longest (k = 0), part p takes k = p, 2 parts - 1 - p,
// 2 parts + p, 4 parts - 1 - p, ...: a long block is paired with a short one, so the parts carry
// nearly equal work. Returns false when part `part` has no it-th block.
__host__ __device__ __forceinline__ bool block_at(int it, int part, int parts, int n, Block* bk) {
  const int nblk = (n + 2 * kTile - 1) / (2 * kTile);
  const int k = 2 * parts * (it >> 1) + ((it & 1) ? 2 * parts - 1 - part : part);
  if (k >= nblk) return false;
  *bk = block_of(nblk - 1 - k, n);
  return true;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
               PrefillArgs a, int parts) {
  extern __shared__ uint8_t smem_raw[];
  AttnSmem& sm = *reinterpret_cast<AttnSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

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
      mbar_init(&sm.k_empty[i], 2);
      mbar_init(&sm.v_full[i], 1);
      mbar_init(&sm.v_empty[i], 2);
      for (int bf = 0; bf < 2; ++bf) {
        mbar_init(&sm.s_full[i][bf], 1);
        mbar_init(&sm.p_ready[i][bf], kTile);
        mbar_init(&sm.o_done[i][bf], 1);
      }
    }
    mbar_init(&sm.stage_free, 1);
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

  if (warp == kSoftmaxWarps + 2) {
    // ---------------------------------------------------------------- TMA loads
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      bool ok = true;
      int kv = 0;                                      // K/V tiles loaded so far (stage = kv & 1)
      int nq[2] = {0, 0};                              // Q loads issued per tile
      for (int it = 0; ok; ++it) {
        Block bk;
        if (!block_at(it, part, parts, n, &bk)) break;   // longest block first
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
        // Key tiles go up in even blocks and down in odd ones: the tiles a block read last are the
        // first ones the next block reads, so they are still in L2 (always going up evicts them all).
        const bool down = it & 1;
        for (int jj = 0; jj < bk.nkt && ok; ++jj, ++kv) {
          const int j = down ? bk.nkt - 1 - jj : jj;
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
  } else if (warp >= kSoftmaxWarps) {
    // ---------------------------------------------------------------- MMA issue, one thread per tile
    const int w = warp - kSoftmaxWarps;
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(kTile, kHalf, false, false);   // S = Q K^T (64 keys), both K-major
      constexpr uint32_t idesc_o = idesc_bf16(kTile, kTile, false, true);    // O += P V, V is MN-major
      // operand descriptors are built once; a k-step only adds a constant to the start-address field
      const uint64_t dq = smem_desc_sw128(smem_u32(sm.q[w]), 16, 1024);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, 1024), dk1 = smem_desc_sw128(smem_u32(sm.k[1]), 16, 1024);
      const uint64_t dv0 = smem_desc_sw128(smem_u32(sm.v[0]), kHalfBytes, 1024);
      const uint64_t dv1 = smem_desc_sw128(smem_u32(sm.v[1]), kHalfBytes, 1024);
      const uint32_t t_base = tmem + w * 256, o_tmem = t_base + 128;
      bool ok = true;
      int kvu = 0;   // K/V tiles of the ring that earlier blocks used
      int nq = 0;    // Q loads of this tile consumed
      int hs = 0;    // half-steps of this tile done in earlier blocks (even)
      for (int it = 0; ok; ++it) {
        Block bk;
        if (!block_at(it, part, parts, n, &bk)) break;
        const int nkt_w = w ? bk.nkt1 : bk.nkt0;
        const int T = 2 * nkt_w;
        // when the key tiles come in descending order, the one tile 0 does not read comes first
        const int skip = ((it & 1) && nkt_w && nkt_w < bk.nkt) ? 1 : 0;
        // K/V tile `ring` of the CTA's load sequence is not read by this tile: wait until it has
        // landed (which also means the phase before it is closed), then release it
        auto release = [&](int ring) {
          const int st = ring & 1, par = (ring >> 1) & 1;
          ok = mbar_wait(&sm.k_full[st], par, abort_flag, a.status, code);
          if (ok) mbar_arrive(&sm.k_empty[st]);
          if (ok) ok = mbar_wait(&sm.v_full[st], par, abort_flag, a.status, code);
          if (ok) mbar_arrive(&sm.v_empty[st]);
        };
        // S(t): keys 64 t .. 64 t + 63 = rows (t & 1) * 64 .. of K tile t / 2, into S buffer t & 1
        auto issue_s = [&](int t) {
          const int ring = kvu + skip + (t >> 1), st = ring & 1, bf = t & 1;
          if (bf == 0) {
            ok = mbar_wait(&sm.k_full[st], (ring >> 1) & 1, abort_flag, a.status, code);
            if (!ok) return;
            tc_fence_after();
          }
          const uint64_t kd = (st ? dk1 : dk0) + (uint64_t)((bf * kHalf * 128) >> 4);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
            mma_ss(t_base + bf * kHalf, dq + off, kd + off, idesc_s, kk > 0);
          }
          mma_commit(&sm.s_full[w][bf]);
          if (bf == 1) mma_commit(&sm.k_empty[st]);
          if (t == T - 1) mma_commit(&sm.q_empty[w]);     // last read of this block's Q tile
        };
        if (T == 0) {
          for (int j = 0; j < bk.nkt && ok; ++j) release(kvu + j);
          kvu += bk.nkt;
          continue;
        }
        if (skip) release(kvu);
        if (ok) ok = mbar_wait(&sm.q_full[w], nq & 1, abort_flag, a.status, code);
        ++nq;
        if (ok) issue_s(0);
        if (ok) issue_s(1);
        for (int t = 0; t < T && ok; ++t) {
          const int ring = kvu + skip + (t >> 1), st = ring & 1, bf = t & 1;
          if (bf == 0) ok = mbar_wait(&sm.v_full[st], (ring >> 1) & 1, abort_flag, a.status, code);
          if (ok) ok = mbar_wait(&sm.p_ready[w][bf], ((hs + t) >> 1) & 1, abort_flag, a.status, code);
          if (!ok) break;
          tc_fence_after();
          const uint64_t vd = (st ? dv1 : dv0) + (uint64_t)((bf * kHalf * 128) >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)   // 16 keys per step: 8 TMEM columns of P, 16 rows of V
            mma_ts(o_tmem, t_base + bf * kHalf + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), idesc_o,
                   (t > 0 || kk > 0) ? 1u : 0u);
          if (t >= T - 2) mma_commit(&sm.o_done[w][bf]);   // the block's last two PVs: one phase per block each
          if (bf == 1) mma_commit(&sm.v_empty[st]);
          if (t + 2 < T) issue_s(t + 2);
        }
        if (ok && nkt_w < bk.nkt && !skip) release(kvu + bk.nkt - 1);   // tile 1's diagonal K/V tile
        kvu += bk.nkt;
        hs += T;
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- softmax, thread = query row
    const int w = warp >> 2;
    const int row = threadIdx.x & (kTile - 1);
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_base = tmem + lane_base + w * 256;
    const uint32_t o_addr = t_base + 128;
    const float sc2 = a.scale * kLog2e;
    bool ok = true;
    int hs = 0;    // half-steps of this tile done in earlier blocks (even)
    int nb = 0;                  // blocks this tile has finished
    int ep_base = 0;             // epilogues of earlier blocks
    bool release_due = false;    // (thread 0 of the tile) its stores may still be reading the staging tile
    for (int it = 0; ok; ++it) {
      Block bk;
      if (!block_at(it, part, parts, n, &bk)) break;
      const int T = 2 * (w ? bk.nkt1 : bk.nkt0);
      if (T == 0) {
        ep_base += 1;
        continue;
      }
      const int i = bk.r0 + w * kTile + row;             // query row of this thread
      float m_used = -INFINITY, l = 0.f;
      for (int t = 0; t < T && ok; ++t) {
        const int bf = t & 1;
        const uint32_t s_addr = t_base + bf * kHalf;
        ok = mbar_wait(&sm.s_full[w][bf], ((hs + t) >> 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        uint32_t s[64];
        tmem_ld32(s_addr, s);
        tmem_ld32(s_addr + 32, s + 32);
        tmem_wait_ld();
        // key tile of this half-step: they come in ascending order in even blocks, descending in odd ones
        const int kt = (it & 1) ? (T >> 1) - 1 - (t >> 1) : (t >> 1);
        if (kt == (T >> 1) - 1) {         // inside the diagonal key tile: key 128 kt + 64 (t & 1) + col is visible iff col <= lim
          const int lim = i - (kt * kTile + (t & 1) * kHalf);
#pragma unroll
          for (int col = 0; col < 64; ++col)
            if (col > lim) s[col] = 0xff800000u;   // -inf
        }
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int col = 0; col < 64; col += 8) {
          mx0 = max3(mx0, __uint_as_float(s[col]), __uint_as_float(s[col + 1]));
          mx1 = max3(mx1, __uint_as_float(s[col + 2]), __uint_as_float(s[col + 3]));
          mx2 = max3(mx2, __uint_as_float(s[col + 4]), __uint_as_float(s[col + 5]));
          mx3 = max3(mx3, __uint_as_float(s[col + 6]), __uint_as_float(s[col + 7]));
        }
        // (-inf when every key of this half-step is hidden from the row: then nothing changes and P = 0)
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sc2;
        const bool need = mx > m_used + kRescaleStep;      // also true on the first half-step (m_used = -inf)
        if (t > 0 && __any_sync(0xffffffffu, need)) {
          // O may be rescaled once it holds every PV up to PV(t-1), the last one these threads have
          // fed. The issuing thread runs S(t+1) right after PV(t-1) and the pipe keeps that order,
          // so S(t+1) having landed is the signal (its barrier is one phase ahead of what this
          // thread has consumed, so the parity wait is valid); the block's last PVs have their own.
          if (t + 1 < T) ok = mbar_wait(&sm.s_full[w][(t + 1) & 1], ((hs + t + 1) >> 1) & 1, abort_flag, a.status, code);
          else ok = mbar_wait(&sm.o_done[w][0], nb & 1, abort_flag, a.status, code);
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
          tmem_st16(s_addr + ch * 16, p);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&sm.p_ready[w][bf]);
        l += (part[0] + part[1]) + (part[2] + part[3]);
        if (release_due) {       // only ever set in thread 0 of the tile
          bulk_wait_read_all();
          mbar_arrive(&sm.stage_free);
          release_due = false;
        }
      }
      // epilogue of the block; the next block's first PV cannot start before these threads have
      // delivered its P(0), i.e. after they are done reading O here
      if (ok) ok = mbar_wait(&sm.o_done[w][1], nb & 1, abort_flag, a.status, code);
      if (!ok) break;
      tc_fence_after();
      // O leaves through shared memory and two TMA stores (rows past n are clipped by the store).
      // The epilogue before this one (the other tile's, or this tile's of the previous block when
      // that block had one tile) must have been read out of the staging tile first.
      if (i < n) a.lse[((int64_t)b * a.Hq + h) * n + i] = (m_used + log2f(l)) * kLn2;
      const float inv = 1.f / l;
      const int seq = ep_base + w;
      if (seq > 0) {
        ok = mbar_wait(&sm.stage_free, (seq - 1) & 1, abort_flag, a.status, code);
        if (!ok) break;
      }
      uint8_t* my_row = sm.o_stage + row * 128;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t o[64];
        tmem_ld32(o_addr + hf * 64, o);
        tmem_ld32(o_addr + hf * 64 + 32, o + 32);
        tmem_wait_ld();
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
      if (w == 0) asm volatile("bar.sync 1, 128;" ::: "memory");   // the 128 threads of this tile
      else asm volatile("bar.sync 2, 128;" ::: "memory");
      if (row == 0) {
        tma_store_4d(&map_o, sm.o_stage, 0, h, bk.r0 + w * kTile, b);
        tma_store_4d(&map_o, sm.o_stage + kHalfBytes, 64, h, bk.r0 + w * kTile, b);
        bulk_commit();
        if (w == 0) {         // tile 0 runs ahead of tile 1 and would wait for its next K tile anyway
          bulk_wait_read_all();
          mbar_arrive(&sm.stage_free);
        } else {
          release_due = true; // signalled a little later, off the path to the next block's first P
        }
      }
      hs += T;
      ++nb;
      ep_base += bk.nkt1 ? 2 : 1;
    }
    if (release_due) {
      bulk_wait_read_all();
      mbar_arrive(&sm.stage_free);
    }
    if (row == 0) bulk_wait_all();   // the last stores have left shared memory and are complete
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
  const size_t smem = sizeof(AttnSmem) + 1024;
  cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // One CTA per (sequence, head) when that fills the SMs evenly; otherwise deal each head's blocks
  // to 2, 4 or 8 CTAs. Cost model: waves of CTAs x the largest share of key-tile steps a CTA gets
  // (a block costs about one step more, a CTA about two); splitting must win by 5 % to be chosen.
  int dev = 0, sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int nblk = (a.n + 2 * kTile - 1) / (2 * kTile);
  const long long heads = (long long)a.Hq * a.B;
  int parts = 1;
  long long best = -1;
  for (int p = 1; p <= 8 && p <= nblk; p *= 2) {
    long long share = 0;                       // key-tile steps of the busiest part
    for (int part = 0; part < p; ++part) {
      long long w = 0;
      Block bk;
      for (int it = 0; block_at(it, part, p, a.n, &bk); ++it) w += bk.nkt + 1;
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
