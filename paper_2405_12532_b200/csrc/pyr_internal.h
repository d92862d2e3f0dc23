// Internal declarations shared by the host dispatcher and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pyr.h"

namespace pyr {

constexpr int kStatusWords = 64;
constexpr int kMaxPrompt = 32768;      // select keeps one sequence's scores in shared memory
constexpr int kMaxDecodeSplits = 64;

// One layer's attention + score problem.
struct PrefillArgs {
  const void* q; const void* k; const void* v; void* out;
  float* lse;          // [B, Hq, n]
  float* score;        // [B, G, c] pooled
  const float* w;      // [L] device
  int64_t qsb, qsn, qsh, ksb, ksn, ksh, osb, osn, osh;
  int B, n, Hq, Hkv, D, L, G;   // L = window actually present (min(L, n)); c = n - L
  float scale;
  int dtype;
  int* status;
  // select-first ordering (tcgen05 path): only the query tiles k0 <= k < k1, numbered from the last (longest) tile,
  // are computed; with `rank` ([B, G, n]: a row's place among the kept rows of its selection group, -1 if dropped)
  // every output row goes to its place instead of its own row
  int tile_k0 = 0, tile_k1 = 1 << 30;
  const int32_t* rank = nullptr;
};

struct SelectArgs {
  const float* score;  // [B, G, c]
  int32_t* idx;        // [B, G, n_out]
  const int32_t* pos_in;   // [B, G, n] or nullptr = identity
  int32_t* pos_out;    // [B, G, n_out]
  int B, G, n, c, k;   // n_out = k + (n - c)
  int reencode = 0;    // 1: positions are re-encoded from 0 in kept order instead of gathered
  int32_t* rank = nullptr;   // [B, G, n] or nullptr: the inverse of idx (-1 for dropped rows)
};

struct GatherArgs {
  const void* k; const void* v;    // [B, n, Hkv, D] strided
  void* kc; void* vc;              // [B, Hkv, cap, D]
  const int32_t* idx;              // [B, G, n_out]
  int64_t ksb, ksn, ksh;
  int B, Hkv, G, D, n_out, cap, elem_bytes;
};

struct RowsArgs {
  void* rows; const int32_t* idx;
  int64_t stride_b, stride_n, stride_g;   // elements
  int64_t row_elems;
  int B, G, n_out, elem_bytes;
  int idx_div;         // consecutive row groups that share one index list (1: a list per group)
  int dst_begin = 0;   // rows below this destination, and rows whose source lies below src_begin, are in place already
  int src_begin = 0;
};

// Generation-phase score of a layer's cache from its window of recent queries.
struct GenScoreArgs {
  const void* qwin;    // [B, R, Hq, D]: ring of the most recent queries; window query i is slot (start + i) % R
  const void* kc;      // [B, Hkv, cap, D]
  float* part;         // [B, Hq, query tiles, c] per-head partial scores
  float* score;        // [B, G, c] pooled
  const float* w;      // [Lw] device, oldest first
  int B, Hq, Hkv, D, G, R, start, Lw, len, cap, c;   // c = len - Lw context rows
  float scale;
  int dtype;
};

struct DecodeArgs {
  const void* q; const void* k_new; const void* v_new; void* out;
  void* kc; void* vc;              // [B, Hkv, cap, D]
  float* part_acc;                 // [B, Hq, splits, D]
  float* part_ml;                  // [B, Hq, splits, 2]
  int B, Hq, Hkv, D, len, cap, splits, rows_per_split;   // len = rows before the append
  float scale;
  int dtype;
  int* status;                     // device status word, may be null
  uint32_t spin_limit = 0;         // iterations a device-side wait may spin; 0 = the default
  int skip_chunk = -1;                // -1; else the loader leaves this chunk of every split out (exercises the waits' failure path)
};

// Split-K rule of the decode kernels: rows [0, total) of a cache are cut into `splits` ranges of
// `rows_per_split` (a multiple of 16) so that the grid is at most one wave of two CTAs per SM when
// splitting is needed at all. The kernels are bandwidth-bound and every CTA pays about 5 us of
// set-up and merging: a second, partial wave costs that again (measured: 13 us per launch).
inline void decode_split_rule(int batch, int n_kv_heads, int total, int sms, int* splits_out, int* rows_per_split_out) {
  const long long pairs = (long long)batch * n_kv_heads;
  int splits = (int)(((long long)sms * 2) / pairs);
  const int max_by_rows = (total + 127) / 128;
  if (splits > max_by_rows) splits = max_by_rows;
  if (splits > kMaxDecodeSplits) splits = kMaxDecodeSplits;
  if (splits < 1) splits = 1;
  int rps = (total + splits - 1) / splits;
  rps = (rps + 15) / 16 * 16;
  *splits_out = (total + rps - 1) / rps;
  *rows_per_split_out = rps;
}

// Multiprocessors of the current device (asked once per device; 0 if the query fails).
int device_sm_count();
// Adds to the count that pyr_launch_count reports.
void count_launches(int kernels);

cudaError_t launch_prefill_simt(const PrefillArgs& a, cudaStream_t s);
cudaError_t launch_score_simt(const PrefillArgs& a, cudaStream_t s);
cudaError_t launch_prefill_tc(const PrefillArgs& a, cudaStream_t s);     // bf16, D = 128, tcgen05
// `partial` holds B * Hq * score_tc_chunks(L) * score_tc_groups() * c floats: per-head partial scores, summed by a second kernel
cudaError_t launch_score_tc(const PrefillArgs& a, float* partial, cudaStream_t s);
int score_tc_chunks(int L);
int score_tc_groups();
bool prefill_tc_supported(const PrefillArgs& a);
bool score_tc_supported(const PrefillArgs& a);
cudaError_t launch_select(const SelectArgs& a, cudaStream_t s);
cudaError_t launch_gather_kv(const GatherArgs& a, cudaStream_t s);
cudaError_t launch_compact_rows(const RowsArgs& a, cudaStream_t s);
cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t s);
// decoder glue of whole-model workloads (csrc/glue.cu); matrices row-major, w is [N, K] (out, in)
cudaError_t launch_glue_embed(const int32_t* ids, const void* table, void* out, int64_t tokens, int d, int vocab,
                              int dtype, int* status, cudaStream_t s);
// Rows of a [batch, n_src, *] tensor picked by a list per sequence: logical row b * n_dst + i is physical row
// b * n_src + rows[b * rows_stride + i]. rows == nullptr: the identity.
struct RowMap {
  const int32_t* rows = nullptr;
  int64_t rows_stride = 0;
  int n_src = 0, n_dst = 1;
#ifdef __CUDACC__
  __host__ __device__
#endif
  int64_t source_row(int64_t m) const {
    if (!rows) return m;
    const int64_t b = m / n_dst;
    return b * n_src + rows[b * rows_stride + (m - b * n_dst)];
  }
};
cudaError_t launch_glue_rmsnorm(const void* x, const void* gain, void* out, int64_t tokens, int d, float eps, int dtype,
                                const RowMap& map, cudaStream_t s);
cudaError_t launch_glue_linear(const void* x, const void* w, const void* res, void* y, int64_t M, int N, int K, int dtype,
                               const RowMap& map, cudaStream_t s);
// bf16 tensor-core GEMM of the glue (csrc/gemm_tc.cu): y = x w^T (+ res); w is [N, K]
bool gemm_tc_supported(const void* x, const void* w, const void* res, const void* y, int64_t M, int N, int K);
cudaError_t launch_gemm_tc(const void* x, const void* w, const void* res, void* y, int64_t M, int N, int K, int* status,
                           const RowMap& res_map, cudaStream_t s);
cudaError_t launch_gemm_tc_gated(const void* x, const void* wg, const void* wu, void* out, int64_t M, int N, int K,
                                 int* status, cudaStream_t s);
int* glue_status_word();     // the current GPU's status word of the glue GEMMs (null if it cannot be resolved)
bool gemm_skinny_supported(const void* x, const void* w, const void* res, const void* y, int64_t M, int N, int K);
// y may be given as up to four column parts ys[i] of [M, N / n_parts] each (n_parts > 1: no residual, parts of whole 128s)
cudaError_t launch_gemm_skinny(const void* x, const void* w, const void* res, void* const* ys, int n_parts, int64_t M, int N,
                               int K, int* status, cudaStream_t s);
cudaError_t launch_glue_rope(void* x, const int32_t* pos, int64_t tokens, int H, int D, int dtype, cudaStream_t s);
cudaError_t launch_glue_swiglu(const void* g, const void* u, void* out, int64_t n, int dtype, cudaStream_t s);
cudaError_t launch_glue_argmax(const void* x, int32_t* out, int64_t rows, int n, int dtype, cudaStream_t s);
int gen_score_qtiles(int Lw);
cudaError_t launch_gen_score(const GenScoreArgs& a, cudaStream_t s);     // two kernels
// rows of row_bytes (a multiple of 16) per batch entry, byte strides
cudaError_t launch_copy_rows(const void* src, void* dst, int64_t src_sb, int64_t src_sn, int64_t dst_sb,
                             int64_t dst_sn, int B, int rows, int row_bytes, cudaStream_t s);

}  // namespace pyr
