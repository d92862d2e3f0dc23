// Algorithm 1: "TopP_index <- TopP(A_e, p)" and "PvC <- Gather(KV, TopP_index)".
//
// The paper attributes the added cost of the method to the sort inside top-p
// (Appendix A.1). A selection needs no order among the kept keys, so the
// k-th largest score is found by a most-significant-digit radix select over
// the score bit patterns held in shared memory, and the kept set is written in
// ascending index order by a block-wide prefix count. Equal scores at the cut
// go to the lower indices.
#include "pyr_internal.h"

namespace pyr {
namespace {


// Order-preserving map from float bits to unsigned (larger float -> larger key).
__device__ __forceinline__ uint32_t float_key(float x) {
  uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One CTA per (sequence, selection group). kSelThreads = 1024 for a few long selections, 256 when
// there are many (more CTAs per SM at once: the kernel is bound by its barriers, not by its data).
template <int kSelThreads>
__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectArgs a) {
  extern __shared__ uint32_t keys[];       // [c]
  __shared__ uint32_t hist[256];
  __shared__ uint32_t warp_tot[kSelThreads / 32];
  __shared__ uint32_t sh_prefix, sh_remaining, sh_running;

  const int bg = blockIdx.x;
  const int t = threadIdx.x;
  const int c = a.c, k = a.k, n = a.n;
  const int window = n - c;
  const int n_out = k + window;
  int32_t* idx = a.idx + (int64_t)bg * n_out;
  int32_t* pos_out = a.pos_out + (int64_t)bg * n_out;
  const int32_t* pos_in = a.pos_in ? a.pos_in + (int64_t)bg * n : nullptr;
  int32_t* rank = a.rank ? a.rank + (int64_t)bg * n : nullptr;

  // the window is always kept
  for (int i = t; i < window; i += kSelThreads) {
    idx[k + i] = c + i;
    pos_out[k + i] = a.reencode ? k + i : (pos_in ? pos_in[c + i] : c + i);
    if (rank) rank[c + i] = k + i;
  }
  if (k == 0) {
    if (rank) for (int i = t; i < c; i += kSelThreads) rank[i] = -1;
    return;
  }
  if (k == c) {
    for (int i = t; i < c; i += kSelThreads) {
      idx[i] = i;
      pos_out[i] = a.reencode ? i : (pos_in ? pos_in[i] : i);
      if (rank) rank[i] = i;
    }
    return;
  }
  const float* score = a.score + (int64_t)bg * c;
  for (int i = t; i < c; i += kSelThreads) keys[i] = float_key(score[i]);
  if (t == 0) { sh_prefix = 0; sh_remaining = (uint32_t)k; }
  __syncthreads();

  // Four 8-bit digits, most significant first. After the passes sh_prefix is
  // the key of the k-th largest score and sh_remaining how many keys equal to
  // it are kept.
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t hi_mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
    if (t < 256) hist[t] = 0;
    __syncthreads();
    const uint32_t prefix = sh_prefix;
    for (int i = t; i < c; i += kSelThreads) {
      uint32_t key = keys[i];
      if ((key & hi_mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (t < 32) {
      // warp 0 walks the 256 bins from the top, 8 bins per lane
      const uint32_t rem = sh_remaining;   // read by every lane before the shuffles below
      uint32_t local[8], sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { local[j] = hist[255 - (t * 8 + j)]; sum += local[j]; }
      uint32_t incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
        if (t >= o) incl += y;
      }
      const uint32_t excl = incl - sum;
      if (excl < rem && rem <= incl) {      // the k-th largest falls in this lane's bins
        uint32_t run = excl;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (run < rem && rem <= run + local[j]) {
            sh_prefix = prefix | ((uint32_t)(255 - (t * 8 + j)) << shift);
            sh_remaining = rem - run;
          }
          run += local[j];
        }
      }
    }
    __syncthreads();
  }
  const uint32_t tau = sh_prefix;
  const uint32_t need_eq = sh_remaining;
  if (t == 0) sh_running = 0;
  __syncthreads();

  // Ascending write-out. Counts of (greater, equal) before each element are
  // packed as (gt << 16 | eq); c <= 32768 keeps both halves in range.
  const int lane = t & 31, warp = t >> 5;
  for (int base = 0; base < c; base += kSelThreads) {
    const int i = base + t;
    uint32_t key = i < c ? keys[i] : 0u;
    const bool gt = i < c && key > tau;
    const bool eq = i < c && key == tau;
    const uint32_t bgt = __ballot_sync(0xffffffffu, gt);
    const uint32_t beq = __ballot_sync(0xffffffffu, eq);
    const uint32_t below = (1u << lane) - 1u;
    uint32_t mine = ((uint32_t)__popc(bgt & below) << 16) | (uint32_t)__popc(beq & below);
    if (lane == 0) warp_tot[warp] = ((uint32_t)__popc(bgt) << 16) | (uint32_t)__popc(beq);
    __syncthreads();
    uint32_t before = sh_running;
    for (int wI = 0; wI < warp; ++wI) before += warp_tot[wI];
    before += mine;
    const uint32_t gt_before = before >> 16, eq_before = before & 0xFFFFu;
    const bool keep = gt || (eq && eq_before < need_eq);
    if (keep) {
      const uint32_t p = gt_before + min(eq_before, need_eq);
      idx[p] = i;
      pos_out[p] = a.reencode ? (int)p : (pos_in ? pos_in[i] : i);
      if (rank) rank[i] = (int)p;
    } else if (rank && i < c) {
      rank[i] = -1;
    }
    __syncthreads();
    if (t == kSelThreads - 1) sh_running = before + (gt ? (1u << 16) : 0u) + (eq ? 1u : 0u);
    __syncthreads();
  }
}

// K/V gather into the layer cache: 16 bytes per thread, consecutive threads
// cover one row, then the next kept row of the same (sequence, KV head).
template <int UNROLL>
__global__ void __launch_bounds__(256) gather_kv_kernel(GatherArgs a, int lanes_per_row, int64_t total) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t e0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int eb = a.elem_bytes;
  const int heads_per_group = a.Hkv / a.G;
  for (; e0 < total; e0 += stride * UNROLL) {
    uint4 kv[UNROLL], vv[UNROLL];
    int64_t dst[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int64_t e = e0 + u * stride;
      dst[u] = -1;
      if (e < total) {
        const int lane = (int)(e % lanes_per_row);
        int64_t r = e / lanes_per_row;
        const int i = (int)(r % a.n_out); r /= a.n_out;
        const int h = (int)(r % a.Hkv);
        const int b = (int)(r / a.Hkv);
        const int src_row = a.idx[((int64_t)b * a.G + h / heads_per_group) * a.n_out + i];
        const int64_t src = ((int64_t)b * a.ksb + (int64_t)src_row * a.ksn + (int64_t)h * a.ksh) * eb + lane * 16;
        kv[u] = *reinterpret_cast<const uint4*>(static_cast<const char*>(a.k) + src);
        vv[u] = *reinterpret_cast<const uint4*>(static_cast<const char*>(a.v) + src);
        dst[u] = (((int64_t)b * a.Hkv + h) * a.cap + i) * (int64_t)a.D * eb + lane * 16;
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (dst[u] >= 0) {
        *reinterpret_cast<uint4*>(static_cast<char*>(a.kc) + dst[u]) = kv[u];
        *reinterpret_cast<uint4*>(static_cast<char*>(a.vc) + dst[u]) = vv[u];
      }
    }
  }
}

// In-place row compaction. Kept indices ascend, so row i of the result comes
// from a row >= i. One CTA owns one column slab of one (sequence, group) and
// walks the kept rows in ascending chunks: read the whole chunk, barrier,
// write it. A chunk's destinations lie below every source of later chunks, so
// nothing unread is overwritten; slabs of different columns never meet.
constexpr int kRowThreads = 256;
constexpr int kRowUnroll = 4;

__global__ void __launch_bounds__(kRowThreads, 4) compact_rows_kernel(RowsArgs a, int slab_lanes, int slabs, int items) {
  // Items (one column slab of one stream) are dealt round-robin to a grid that fits the machine at
  // once: with one CTA per item a last, partly filled wave of CTAs would run at a fraction of the
  // bandwidth.
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
  const int slab = item % slabs;
  const int bg = item / slabs;
  const int b = bg / a.G, g = bg % a.G;
  const int eb = a.elem_bytes;
  const int lanes_total = (int)(a.row_elems * eb / 16);
  const int lane0 = slab * slab_lanes;
  const int lanes = min(slab_lanes, lanes_total - lane0);
  if (lanes <= 0) continue;
  char* base = static_cast<char*>(a.rows) + ((int64_t)b * a.stride_b + (int64_t)g * a.stride_g) * eb + (int64_t)lane0 * 16;
  const int64_t row_bytes = a.stride_n * eb;
  const int32_t* idx = a.idx + ((int64_t)b * (a.G / a.idx_div) + g / a.idx_div) * a.n_out;
  const int rows_per_iter = (kRowThreads * kRowUnroll) / lanes;   // lanes <= kRowThreads
  const int t = threadIdx.x;
  // Chunk i + 1 is read while chunk i is written: the sources of a later chunk lie above every
  // destination of an earlier one, so only the reads and writes of the same chunk need the barrier.
  // (Four CTAs per SM: the few registers this costs in spills are cheaper than a CTA less.)
  uint4 buf[2][kRowUnroll];
  int ln[kRowUnroll], rr[kRowUnroll];
#pragma unroll
  for (int u = 0; u < kRowUnroll; ++u) {
    ln[u] = (u * kRowThreads + t) % lanes;
    rr[u] = (u * kRowThreads + t) / lanes;
  }
  // The kept indices of a chunk are fetched one chunk before its rows are: the row loads then go out without
  // first waiting for an index, and that wait was most of an iteration.
  auto fetch_idx = [&](int r0, int* src) {
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u)
      src[u] = (rr[u] < rows_per_iter && r0 + rr[u] < a.n_out) ? idx[r0 + rr[u]] : -1;
  };
  // returns the mask of this thread's pieces that move (rows already in place are not touched)
  auto read_chunk = [&](int r0, const int* src, uint4* bf) -> uint32_t {
    uint32_t moved = 0;
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u) {
      if (src[u] >= 0 && src[u] != r0 + rr[u] && src[u] >= a.src_begin) {
        moved |= 1u << u;
        bf[u] = *reinterpret_cast<const uint4*>(base + (int64_t)src[u] * row_bytes + ln[u] * 16);
      }
    }
    return moved;
  };
  auto write_chunk = [&](int r0, const uint4* bf, uint32_t moved) {
#pragma unroll
    for (int u = 0; u < kRowUnroll; ++u)
      if (moved & (1u << u)) *reinterpret_cast<uint4*>(base + (int64_t)(r0 + rr[u]) * row_bytes + ln[u] * 16) = bf[u];
  };
  const int first = a.dst_begin / rows_per_iter * rows_per_iter;
  int src_a[kRowUnroll], src_b[kRowUnroll];
  fetch_idx(first, src_a);
  fetch_idx(first + rows_per_iter, src_b);
  uint32_t mv0 = read_chunk(first, src_a, buf[0]), mv1 = 0;
  __syncthreads();
  // The barrier after a chunk's write keeps a fast thread from writing rows a slow one has yet to read. Where every
  // row moves up by at least d rows, a thread may run floor(d / rows per chunk) chunks ahead before that can happen,
  // so the barrier is only taken every so many chunks (d never shrinks along a stream; it is read again at each
  // barrier). Where rows barely move - the start of a stream - that is every chunk, as before.
  int since = 0, every = 1;
  auto barrier_if_due = [&](int r_next) {
    if (++since >= every) {
      __syncthreads();
      since = 0;
      const int at = r_next < a.n_out ? r_next : a.n_out - 1;
      const int ahead = (idx[at] - at) / rows_per_iter;
      every = ahead < 15 ? ahead + 1 : 16;
    }
  };
  for (int r0 = first; r0 < a.n_out; r0 += 2 * rows_per_iter) {
    fetch_idx(r0 + 2 * rows_per_iter, src_a);
    if (r0 + rows_per_iter < a.n_out) mv1 = read_chunk(r0 + rows_per_iter, src_b, buf[1]);
    write_chunk(r0, buf[0], mv0);
    barrier_if_due(r0 + rows_per_iter);
    if (r0 + rows_per_iter >= a.n_out) break;
    fetch_idx(r0 + 3 * rows_per_iter, src_b);
    mv0 = 0;
    if (r0 + 2 * rows_per_iter < a.n_out) mv0 = read_chunk(r0 + 2 * rows_per_iter, src_a, buf[0]);
    write_chunk(r0 + rows_per_iter, buf[1], mv1);
    barrier_if_due(r0 + 2 * rows_per_iter);
  }
  __syncthreads();       // the next item starts from a barrier like the first
  }
}

}  // namespace

cudaError_t launch_select(const SelectArgs& a, cudaStream_t s) {
  const size_t smem = (size_t)(a.c > 0 ? a.c : 1) * sizeof(uint32_t);
  const int sms = device_sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const bool many = (long long)a.B * a.G > 2LL * sms && a.c <= 8192;
  cudaError_t e = many ? cudaFuncSetAttribute(select_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              kMaxPrompt * (int)sizeof(uint32_t))
                       : cudaFuncSetAttribute(select_kernel<1024>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              kMaxPrompt * (int)sizeof(uint32_t));
  if (e != cudaSuccess) return e;
  if (many) select_kernel<256><<<a.B * a.G, 256, smem, s>>>(a);
  else select_kernel<1024><<<a.B * a.G, 1024, smem, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gather_kv(const GatherArgs& a, cudaStream_t s) {
  const int lanes = a.D * a.elem_bytes / 16;
  const int64_t total = (int64_t)a.B * a.Hkv * a.n_out * lanes;
  if (total == 0) return cudaSuccess;
  constexpr int U = 4;
  int64_t blocks = (total + 256 * U - 1) / (256 * U);
  const int sms = device_sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const int64_t cap = (int64_t)sms * 32;
  if (blocks > cap) blocks = cap;
  gather_kv_kernel<U><<<(unsigned)blocks, 256, 0, s>>>(a, lanes, total);
  return cudaGetLastError();
}

cudaError_t launch_compact_rows(const RowsArgs& a, cudaStream_t s) {
  const int lanes_total = (int)(a.row_elems * a.elem_bytes / 16);
  const int sms = device_sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  // A stream (one sequence, one group) is compacted front to back, so what runs in parallel are the
  // streams and the column slabs they are cut into. Slabs of 32 lanes = 512 bytes of a row, narrowed
  // (down to 64 bytes) only while there are fewer items than CTAs the machine holds at once: narrow
  // slabs cost DRAM efficiency (measured: 0.80 -> 0.75 of peak on 8 KB rows), idle SMs cost more.
  const int resident = sms * 4;                 // CTAs of this kernel an SM holds (64 registers x 256 threads)
  int slab_lanes = lanes_total < 32 ? lanes_total : 32;
  while (slab_lanes > 4 && (long long)a.B * a.G * ((lanes_total + slab_lanes - 1) / slab_lanes) < resident)
    slab_lanes /= 2;
  const int slabs = (lanes_total + slab_lanes - 1) / slab_lanes;
  const long long items = (long long)a.B * a.G * slabs;
  const int grid = (int)(items < 2LL * resident ? items : 2LL * resident);
  compact_rows_kernel<<<grid, kRowThreads, 0, s>>>(a, slab_lanes, slabs, (int)items);
  return cudaGetLastError();
}

}  // namespace pyr
