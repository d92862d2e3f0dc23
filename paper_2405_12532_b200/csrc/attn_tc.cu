// tcgen05 causal attention of the prefill step (bf16, head_dim 128):
// Algorithm 1, "compute attention weights of KV", and the attention output.
//
// A CTA owns one (sequence, head), or one of 2, 4 or 8 shares of it when there
// are too few heads to fill the SMs evenly, and walks its 128-row query tiles
// one at a time, longest first (key tiles up in even tiles of the walk and down
// in odd ones, so that a tile starts on K/V still in L2). The K tiles of all
// query tiles form one stream r = 0, 1, 2, ... that every role walks on its own.
//   warps 0-3    softmax group 0, thread = one query row; takes the even r
//   warps 4-7    softmax group 1 (same rows); takes the odd r
//   warp 8       issues the S MMAs:  S(r) = Q K(r)^T, 128 keys, Q and K from shared memory
//   warp 9       TMA loads of Q and K (two stages of K)
//   warp 10      issues the PV MMAs: O += P(r) V(r), P from tensor memory
//   warp 11      TMA loads of V (two stages)
//   warps 12-15  epilogue of every tile: O / row sum -> bf16 -> shared memory -> TMA store, and lse
// Tensor memory (512 columns): S buffers 0 and 1 (128 fp32 columns each), P
// buffers 0 and 1 (64 columns each: 128 bf16), O (128 columns). Group g owns S
// buffer g, P buffer g and their barriers. A softmax thread reads its row's 128
// scores into registers and releases the S buffer at once, so S(r + 2) is
// computed while the exponentials of r are taken; P(r) is written to the P
// buffer once PV(r - 2) has read it. What couples the groups is the maximum
// used in the exponent: the thread of K tile r reads the value published for
// r - 1 (one word per row and tile parity), raises it only when the row maximum
// has grown by more than 2^8 (which keeps rescaling of O, a TMEM round trip,
// rare), and publishes its own before it starts on the exponentials. Each group
// keeps its own row sum and hands it, with the maximum it is relative to, to the
// epilogue warps, which add the two under the final maximum: the result is the
// exact softmax. The softmax groups never wait for a tile to be written out.
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
constexpr int kWarpS = 8, kWarpLoadQK = 9, kWarpPV = 10, kWarpLoadV = 11, kWarpEpi = 12;
constexpr int kThreads = 16 * 32;
constexpr float kRescaleStep = 8.0f;
// kRegsLaunch must be what ptxas reports for the kernel
constexpr int kRegsLaunch = 128, kRegsSoftmax = 208, kRegsIssue = 40, kRegsEpi = 56;
constexpr uint32_t kColP = 256;             // P buffers: columns 256..319 and 320..383
constexpr uint32_t kColO = 384;             // O: columns 384..511
constexpr int kFinSlots = 4;                // tiles whose row sums may be waiting for the epilogue

struct AttnSmem {
  alignas(1024) uint8_t q[2][kTileBytes];
  alignas(1024) uint8_t k[2][kTileBytes];
  alignas(1024) uint8_t v[2][kTileBytes];
  alignas(1024) uint8_t o_stage[kHalfBytes];         // a [128 x 64] bf16 half tile of O on its way out
  unsigned long long m_slot[2][kTile];               // [tile parity][row]: (K tiles decided so far) << 32 | bits of the maximum in use
  unsigned long long fin[2][kFinSlots][kTile];                   // [group][tile % 4][row]: bits of the group's row sum of the tile << 32 | bits of the maximum it is relative to
  uint64_t q_full[2], q_empty[2];                    // per Q buffer
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];   // per stage
  uint64_t s_full[2], s_free[2], p_ready[2], pv_done[2];   // per group: S landed / S is in registers / P written / PV has read P
  uint64_t o_full;                                   // the last PV of a tile is complete
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
// A launch may cover only the tiles k0 <= k < k1 (select-first ordering: the tiles that hold the
// recent window first, the rest once the kept rows are known).
__host__ __device__ __forceinline__ bool tile_at(int it, int part, int parts, int n, int k0, int k1, Tile* tl) {
  const int ntiles = (n + kTile - 1) / kTile;
  const int k = k0 + 2 * parts * (it >> 1) + ((it & 1) ? 2 * parts - 1 - part : part);
  if (k >= ntiles || k >= k1) return false;
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

// Barrier of the 128 threads of one role that also tells every one of them whether any came with `bad`.
template <int kId>
__device__ __forceinline__ bool bar_any(bool bad) {
  uint32_t any;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, %2, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(any) : "r"((uint32_t)(bad ? 1 : 0)), "n"(kId) : "memory");
  return any != 0;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                PrefillArgs a, int parts) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // The tiles need 1024-byte alignment. The launch asks for what the struct needs plus a kilobyte;
  // if the window's base is not aligned well enough for that, the CTA reports it instead of
  // running past the end.
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

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.q_full[i], 1);
      mbar_init(&sm.q_empty[i], 1);
      mbar_init(&sm.k_full[i], 1);
      mbar_init(&sm.k_empty[i], 1);
      mbar_init(&sm.v_full[i], 1);
      mbar_init(&sm.v_empty[i], 1);
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.s_free[i], kTile);
      mbar_init(&sm.p_ready[i], kTile);
      mbar_init(&sm.pv_done[i], 1);
    }
    mbar_init(&sm.o_full, 1);
    mbar_init(&sm.o_free, kTile);
    // an earlier CTA of this launch gave up: the whole CTA leaves together (decided by one thread)
    sm.abort_flag = *reinterpret_cast<volatile int*>(a.status) != 0 ? 2 : 0;
    fence_barrier_init();
  }
  if (threadIdx.x < 2 * kTile) (&sm.m_slot[0][0])[threadIdx.x] = 0ull;
  __syncthreads();
  if (sm.abort_flag == 2) return;
  if (warp == kWarpS) {
    tmem_alloc(&sm.tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const int code = PYR_ERR_TIMEOUT;
  // Register split: the block starts with kThreads x kRegsLaunch registers; the issuing / loading
  // warps and the epilogue warps (one warpgroup each) give registers up, the two softmax
  // warpgroups take them.
  static_assert(256 * kRegsSoftmax + 128 * kRegsIssue + 128 * kRegsEpi <= kThreads * kRegsLaunch,
                "register split exceeds the launch's total");

  if (warp >= kWarpEpi) {
    // ---------------------------------------------------------------- epilogue of every tile
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsEpi));
    const int row = threadIdx.x & (kTile - 1);
    const uint32_t o_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + kColO;
    uint8_t* my_row = sm.o_stage + row * 128;
    bool ok = true, stored = false;
    int ring0 = 0;
    // select-first ordering: rows leave for their place among the kept rows of the head's selection group
    const int32_t* rank = a.rank ? a.rank + ((int64_t)b * a.G + (a.G == 1 ? 0 : h / (a.Hq / a.G))) * n : nullptr;
    __nv_bfloat16* out_bh = static_cast<__nv_bfloat16*>(a.out) + (int64_t)b * a.osb + (int64_t)h * a.osh;
    for (int it = 0;; ++it) {
      Tile tl;
      if (!tile_at(it, part, parts, n, a.tile_k0, a.tile_k1, &tl)) break;
      const int nkt = tl.nkt;
      const int i = tl.r0 + row;
      const int gf = (ring0 + nkt - 1) & 1;               // the group that took the tile's last K tile
      if (ok) ok = mbar_wait(&sm.o_full, it & 1, abort_flag, a.status, code);
      if (bar_any<1>(!ok)) break;
      tc_fence_after();
      // Row sums of both groups, each relative to the maximum in use when the group left the tile;
      // the last K tile's maximum is the final one. (Written before the groups' arrivals for their
      // last P of the tile, which the tile's last PV follows.)
      const unsigned long long f = *reinterpret_cast<volatile unsigned long long*>(&sm.fin[gf][it & (kFinSlots - 1)][row]);
      float l = __uint_as_float((uint32_t)(f >> 32));
      const float m_fin = __uint_as_float((uint32_t)f);
      if (nkt >= 2) {
        const unsigned long long o2 = *reinterpret_cast<volatile unsigned long long*>(&sm.fin[gf ^ 1][it & (kFinSlots - 1)][row]);
        l += __uint_as_float((uint32_t)(o2 >> 32)) * ex2(__uint_as_float((uint32_t)o2) - m_fin);
      }
      if (i < n) a.lse[((int64_t)b * a.Hq + h) * n + i] = (m_fin + log2f(l)) * kLn2;
      const float inv = 1.f / l;

      if (rank) {
        // The row goes to its place among the kept rows, straight from registers: a thread writes whole
        // 128-byte lines of its own row, 16 columns of the accumulator at a time (the epilogue warps are
        // short of registers), and the accumulator is free for the next tile after the last load.
        const int dst = i < n ? rank[i] : -1;
        __nv_bfloat16* orow = out_bh + (int64_t)(dst >= 0 ? dst : 0) * a.osn;
#pragma unroll
        for (int c16 = 0; c16 < 8; ++c16) {
          uint32_t o[16];
          tmem_ld16(o_addr + c16 * 16, o);
          tmem_wait_ld();
          if (c16 == 7) {
            tc_fence_before();
            mbar_arrive(&sm.o_free);
          }
          if (dst >= 0) {
            uint4 lo, hi;
            lo.x = pack_bf16(__uint_as_float(o[0]) * inv, __uint_as_float(o[1]) * inv);
            lo.y = pack_bf16(__uint_as_float(o[2]) * inv, __uint_as_float(o[3]) * inv);
            lo.z = pack_bf16(__uint_as_float(o[4]) * inv, __uint_as_float(o[5]) * inv);
            lo.w = pack_bf16(__uint_as_float(o[6]) * inv, __uint_as_float(o[7]) * inv);
            hi.x = pack_bf16(__uint_as_float(o[8]) * inv, __uint_as_float(o[9]) * inv);
            hi.y = pack_bf16(__uint_as_float(o[10]) * inv, __uint_as_float(o[11]) * inv);
            hi.z = pack_bf16(__uint_as_float(o[12]) * inv, __uint_as_float(o[13]) * inv);
            hi.w = pack_bf16(__uint_as_float(o[14]) * inv, __uint_as_float(o[15]) * inv);
            *reinterpret_cast<uint4*>(orow + c16 * 16) = lo;
            *reinterpret_cast<uint4*>(orow + c16 * 16 + 8) = hi;
          }
        }
      } else {
      // O leaves through shared memory, one [128 x 64] half at a time (rows past n are clipped by the store)
#pragma unroll 1
      for (int hf = 0; hf < 2; ++hf) {
        if (row == 0 && stored) bulk_wait_read_all();      // the store before has read the staging half
        asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
        for (int c32 = 0; c32 < 2; ++c32) {
          uint32_t o[32];
          tmem_ld32(o_addr + hf * 64 + c32 * 32, o);
          tmem_wait_ld();
          if (hf == 1 && c32 == 1) {           // the accumulator is in registers: the next tile may overwrite it
            tc_fence_before();
            mbar_arrive(&sm.o_free);
          }
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {     // 16-byte chunk c of the half row sits at c ^ (row & 7): the 128-byte swizzle
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(o[ch * 8 + 0]) * inv, __uint_as_float(o[ch * 8 + 1]) * inv);
            pk.y = pack_bf16(__uint_as_float(o[ch * 8 + 2]) * inv, __uint_as_float(o[ch * 8 + 3]) * inv);
            pk.z = pack_bf16(__uint_as_float(o[ch * 8 + 4]) * inv, __uint_as_float(o[ch * 8 + 5]) * inv);
            pk.w = pack_bf16(__uint_as_float(o[ch * 8 + 6]) * inv, __uint_as_float(o[ch * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(my_row + (((c32 * 4 + ch) ^ (row & 7)) << 4)) = pk;
          }
        }
        fence_proxy_async();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (row == 0) {
          tma_store_4d(&map_o, sm.o_stage, hf * 64, h, tl.r0, b);
          bulk_commit();
          stored = true;
        }
      }
      }
      ring0 += nkt;
    }
    if (row == 0 && stored) bulk_wait_all();   // the last stores have left shared memory and are complete
  } else if (warp >= kSoftmaxWarps) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssue));
  if (warp == kWarpLoadQK) {
    // ---------------------------------------------------------------- TMA loads of Q and K
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      bool ok = true;
      int kv = 0;                                      // K/V tiles loaded so far (stage = kv & 1)
      // Q of tile `it` goes into buffer it & 1 once the S MMAs of tile it - 2 have read it.
      auto load_q = [&](int it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, a.tile_k0, a.tile_k1, &tl)) return;
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
        if (!tile_at(it, part, parts, n, a.tile_k0, a.tile_k1, &tl)) break;   // longest tile first
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
  } else if (warp == kWarpLoadV) {
    // ---------------------------------------------------------------- TMA loads of V
    // (a thread of their own: a V stage is released by its PV, later than the S MMAs release
    // the K stage, and the K loads must not wait for that)
    if (lane == 0) {
      prefetch_tensormap(&map_v);
      bool ok = true;
      int kv = 0;
      for (int it = 0; ok; ++it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, a.tile_k0, a.tile_k1, &tl)) break;
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
  } else if (warp == kWarpS) {
    // ---------------------------------------------------------------- S MMAs: S(r) = Q K^T for K tile r of the stream
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(kTile, kTile, false, false);   // both K-major
      const uint64_t dq0 = smem_desc_sw128(smem_u32(sm.q[0]), 16, 1024), dq1 = smem_desc_sw128(smem_u32(sm.q[1]), 16, 1024);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(sm.k[0]), 16, 1024), dk1 = smem_desc_sw128(smem_u32(sm.k[1]), 16, 1024);
      bool ok = true;
      int ring = 0;                                    // K tiles so far; buffer and stage ring & 1, phase (ring >> 1) & 1
      for (int it = 0; ok; ++it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, a.tile_k0, a.tile_k1, &tl)) break;
        const int bq = it & 1;
        ok = mbar_wait(&sm.q_full[bq], (it >> 1) & 1, abort_flag, a.status, code);
        const uint64_t dq = bq ? dq1 : dq0;
        for (int j = 0; j < tl.nkt && ok; ++j, ++ring) {
          const int st = ring & 1, ph = (ring >> 1) & 1;
          ok = mbar_wait(&sm.k_full[st], ph, abort_flag, a.status, code);
          // the buffer is free once the softmax threads of K tile ring - 2 hold its scores in registers
          if (ok && ring >= 2) ok = mbar_wait(&sm.s_free[st], ph ^ 1, abort_flag, a.status, code);
          if (!ok) break;
          tc_fence_after();
          const uint64_t kd = st ? dk1 : dk0;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
            mma_ss(tmem + st * kTile, dq + off, kd + off, idesc_s, kk > 0);
          }
          mma_commit(&sm.s_full[st]);
          mma_commit(&sm.k_empty[st]);
          if (j == tl.nkt - 1) mma_commit(&sm.q_empty[bq]);     // last read of this Q tile
        }
      }
    }
    __syncwarp();
  } else if (warp == kWarpPV) {
    // ---------------------------------------------------------------- PV MMAs: O += P(r) V
    if (lane == 0) {
      constexpr uint32_t idesc_o = idesc_bf16(kTile, kTile, false, true);    // V is MN-major
      const uint64_t dv0 = smem_desc_sw128(smem_u32(sm.v[0]), kHalfBytes, 1024);
      const uint64_t dv1 = smem_desc_sw128(smem_u32(sm.v[1]), kHalfBytes, 1024);
      const uint32_t o_tmem = tmem + kColO;
      bool ok = true;
      int ring = 0;
      for (int it = 0; ok; ++it) {
        Tile tl;
        if (!tile_at(it, part, parts, n, a.tile_k0, a.tile_k1, &tl)) break;
        // the first PV of a tile overwrites the accumulator of the tile before it
        if (it >= 1) ok = mbar_wait(&sm.o_free, (it - 1) & 1, abort_flag, a.status, code);
        for (int j = 0; j < tl.nkt && ok; ++j, ++ring) {
          const int st = ring & 1, ph = (ring >> 1) & 1;
          ok = mbar_wait(&sm.v_full[st], ph, abort_flag, a.status, code);
          if (ok) ok = mbar_wait(&sm.p_ready[st], ph, abort_flag, a.status, code);
          if (!ok) break;
          tc_fence_after();
          const uint64_t vd = st ? dv1 : dv0;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)   // 16 keys per MMA: 8 TMEM columns of P, 16 rows of V
            mma_ts(o_tmem, tmem + kColP + st * 64 + kk * 8, vd + (uint64_t)((kk * 2048) >> 4), idesc_o,
                   (j > 0 || kk > 0) ? 1u : 0u);
          mma_commit(&sm.pv_done[st]);
          mma_commit(&sm.v_empty[st]);
          if (j == tl.nkt - 1) mma_commit(&sm.o_full);           // the tile's accumulator is complete
        }
      }
    }
    __syncwarp();
  }
  } else {
    // ---------------------------------------------------------------- softmax, thread = query row
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    const int grp = warp >> 2;                           // takes the K tiles r of the stream with r % 2 == grp
    const int row = threadIdx.x & (kTile - 1);
    const uint32_t t_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t o_addr = t_base + kColO;
    const uint32_t s_addr = t_base + grp * kTile;
    const uint32_t p_addr = t_base + kColP + grp * 64;
    const float sc2 = a.scale * kLog2e;
    bool ok = true;
    int ring0 = 0;               // K tiles of earlier tiles

    for (int it = 0; ok; ++it) {
      Tile tl;
      if (!tile_at(it, part, parts, n, a.tile_k0, a.tile_k1, &tl)) break;
      const int nkt = tl.nkt;
      const int i = tl.r0 + row;                          // query row of this thread
      const int tp = it & 1;
      float m_mine = -INFINITY, l = 0.f;                  // this group's row sum and the maximum it is relative to
      // The groups alternate along the whole stream, so the group that finishes a tile is never the
      // one that the next tile starts with.
      const int j0 = ((ring0 & 1) == grp) ? 0 : 1;
      const int j_last = ((ring0 + nkt - 1) & 1) == grp ? nkt - 1 : nkt - 2;   // this group's last K tile of the tile
      for (int j = j0; j < nkt && ok; j += 2) {
        const int ring = ring0 + j;
        const int ph = (ring >> 1) & 1;
        ok = mbar_wait(&sm.s_full[grp], ph, abort_flag, a.status, code);
        if (!ok) break;
        tc_fence_after();
        uint32_t s[kTile];               // the row's 128 scores (the softmax warps hold the registers for it)
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) tmem_ld32(s_addr + ch * 32, s + ch * 32);
        // While the scores are on their way: the maximum in use after the K tile before this one,
        // from the partner thread of this row. A tile's first K tile starts from -inf and waits for
        // nobody: the word of this tile parity was last read two tiles ago (see the P-buffer wait).
        float m_prev = -INFINITY;
        if (j > 0) ok = slot_wait(&sm.m_slot[tp][row], (uint32_t)ring, &m_prev, abort_flag, a.status, code);
        // key tile of this step: ascending in even tiles of the walk, descending in odd ones
        const int kt = (it & 1) ? nkt - 1 - j : j;
        const bool diag = kt == nkt - 1;    // inside the diagonal key tile key 128 kt + col is visible iff col <= i - 128 kt
        const int lim = i - kt * kTile;
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(&sm.s_free[grp]);      // the scores are in registers: S(ring + 2) may overwrite the buffer
        if (diag) {
#pragma unroll
          for (int col = 0; col < kTile; ++col)
            if (col > lim) s[col] = 0xff800000u;   // -inf
        }
        float mx[8];
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) mx[c8] = max3(__uint_as_float(s[c8 * 2]), __uint_as_float(s[c8 * 2 + 1]), -INFINITY);
#pragma unroll
        for (int col = 16; col < kTile; col += 16) {
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8)
            mx[c8] = max3(mx[c8], __uint_as_float(s[col + c8 * 2]), __uint_as_float(s[col + c8 * 2 + 1]));
        }
        const float mxa = max3(mx[0], mx[1], mx[2]), mxb = max3(mx[3], mx[4], mx[5]);
        const float mxs = max3(max3(mxa, mxb, mx[6]), mx[7], -INFINITY) * sc2;   // finite: column 0 of the tile is visible
        // P(ring) goes to this group's P buffer, which PV(ring - 2) must have read. The wait comes
        // before this thread publishes its maximum, so whoever reads that word knows that PV(ring - 2)
        // is complete. That is what makes three things safe: the partner's parity wait for
        // PV(ring - 1) in the rescale below (it reads the word of ring - 1, so PV(ring - 3), the phase
        // before on that barrier, is complete); reusing a tile parity's word without a wait (a tile's
        // first K tile R publishes after PV(R - 2), which needed the P of every K tile of the tile
        // two back, written after their threads read the word); and reusing a row-sum slot four
        // tiles on (PV(R - 2) is then past the first PV of the tile after the slot's, which waited
        // for the epilogue to read it).
        if (ok && ring >= 2) ok = mbar_wait(&sm.pv_done[grp], ph ^ 1, abort_flag, a.status, code);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const bool need = mxs > m_prev + kRescaleStep;      // always true on the first K tile of a tile
        const float m_used = need ? mxs : m_prev;
        *reinterpret_cast<volatile unsigned long long*>(&sm.m_slot[tp][row]) =
            ((unsigned long long)(uint32_t)(ring + 1) << 32) | __float_as_uint(m_used);
        if (j > 0 && __any_sync(0xffffffffu, need)) {
          // O may be rescaled once PV(ring - 1), the other group's, is complete: one phase behind at
          // most (see above), and PV(ring + 1) cannot complete before this thread has written P(ring).
          ok = mbar_wait(&sm.pv_done[grp ^ 1], ((ring - 1) >> 1) & 1, abort_flag, a.status, code);
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
        // P = exp2(S - m) as bf16
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
          tmem_st16(p_addr + ch * 16, p);
        }
        l += (part4[0] + part4[1]) + (part4[2] + part4[3]);
        // The group's row sum of the tile goes to the epilogue warps before the arrival for its last
        // P of the tile: the tile's last PV, which the epilogue waits for, follows that arrival.
        if (j == j_last)
          *reinterpret_cast<volatile unsigned long long*>(&sm.fin[grp][it & (kFinSlots - 1)][row]) =
              ((unsigned long long)__float_as_uint(l) << 32) | __float_as_uint(m_mine);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&sm.p_ready[grp]);
      }
      if (!ok) break;
      ring0 += nkt;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kWarpS) {
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
  const size_t smem = kSmemNeed + 1024;
  if (smem > (size_t)smem_max) return cudaErrorInvalidConfiguration;
  e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // One CTA per (sequence, head) when that fills the SMs evenly; otherwise deal each head's tiles
  // to 2, 4 or 8 CTAs. Cost model: waves of CTAs x the largest share of key-tile steps a CTA gets
  // (a tile costs about one step more, a CTA about two); splitting must win by 5 % to be chosen.
  const int all_tiles = (a.n + kTile - 1) / kTile;
  const int ntiles = (a.tile_k1 < all_tiles ? a.tile_k1 : all_tiles) - a.tile_k0;    // tiles of this launch
  if (ntiles <= 0) return cudaSuccess;
  const long long heads = (long long)a.Hq * a.B;
  int parts = 1;
  long long best = -1;
  for (int p = 1; p <= 8 && p <= ntiles; p *= 2) {
    long long share = 0;                       // key-tile steps of the busiest part
    for (int part = 0; part < p; ++part) {
      long long w = 0;
      Tile tl;
      for (int it = 0; tile_at(it, part, p, a.n, a.tile_k0, a.tile_k1, &tl); ++it) w += tl.nkt + 1;
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
