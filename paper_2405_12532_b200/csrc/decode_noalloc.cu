// pyr_decode_attn_noalloc: the split-K decode attention for callers that must
// not allocate device memory. The split partials, which pyr_decode_attn keeps
// in the workspace of the caller's cache buffer, live here in a fixed array
// that is part of the loaded library image.
#include <mutex>

#include "pyr_internal.h"

namespace {

// 4 MiB of partial results: B * Hq * splits * (D + 2) floats must fit.
constexpr size_t kScratchFloats = (size_t)1 << 20;
static __device__ __align__(256) float g_decode_scratch[kScratchFloats];
// Where a bounded device-side wait of these calls records that it ran out (0 = none did).
static __device__ int g_noalloc_status;

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {};
int* g_status_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// The array's name is only a host-side handle for the symbol. Its device
// address differs per GPU and has to be asked for with that GPU current.
pyr_status_t scratch_for_current_device(float** out, int** status) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return PYR_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return PYR_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev] || !g_status_ptr[dev]) {
    float* p = nullptr;
    int* w = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_decode_scratch) != cudaSuccess || !p)
      return PYR_ERR_CUDA;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&w), g_noalloc_status) != cudaSuccess || !w)
      return PYR_ERR_CUDA;
    g_scratch_ptr[dev] = p;
    g_status_ptr[dev] = w;
  }
  *out = g_scratch_ptr[dev];
  *status = g_status_ptr[dev];
  return PYR_OK;
}

}  // namespace

extern "C" pyr_status_t pyr_decode_attn_noalloc(const void* q, const void* k_new, const void* v_new, void* out,
                                                void* k_cache, void* v_cache, int32_t batch, int32_t n_q_heads,
                                                int32_t n_kv_heads, int32_t head_dim, int32_t dtype, int32_t len,
                                                int32_t cap, float softmax_scale, void* stream) {
  if (!q || !k_new || !v_new || !out || !k_cache || !v_cache) return PYR_ERR_NULL;
  if (batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || len < 0 || cap < 1 ||
      !(softmax_scale >= 0.0f))
    return PYR_ERR_INVALID;
  if (head_dim != 64 && head_dim != 128) return PYR_ERR_UNSUPPORTED;
  if (dtype != PYR_BF16 && dtype != PYR_F32) return PYR_ERR_UNSUPPORTED;
  if (len >= cap) return PYR_ERR_CAPACITY;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
       reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(k_cache) |
       reinterpret_cast<uintptr_t>(v_cache)) % 16)
    return PYR_ERR_INVALID;

  pyr::DecodeArgs a;
  a.q = q; a.k_new = k_new; a.v_new = v_new; a.out = out;
  a.kc = k_cache; a.vc = v_cache;
  a.B = batch; a.Hq = n_q_heads; a.Hkv = n_kv_heads; a.D = head_dim;
  a.len = len; a.cap = cap; a.dtype = dtype;
  a.scale = softmax_scale > 0.0f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
  // same split rule as pyr_decode_attn
  const int sms = pyr::device_sm_count();
  if (sms <= 0) return PYR_ERR_CUDA;
  int splits = 1, rps = 0;
  pyr::decode_split_rule(batch, n_kv_heads, len + 1, sms, &splits, &rps);
  a.splits = splits; a.rows_per_split = rps;

  // The addresses are looked up on every device's first call, whatever its split count: a later
  // call (perhaps inside a stream capture) must not be the one that makes the runtime call.
  float* base = nullptr;
  int* status_word = nullptr;
  pyr_status_t st = scratch_for_current_device(&base, &status_word);
  if (st != PYR_OK) return st;
  a.part_acc = nullptr; a.part_ml = nullptr;
  a.status = status_word;
  a.spin_limit = 0; a.skip_chunk = -1;
  if (splits > 1) {
    const size_t acc_floats = (size_t)batch * n_q_heads * splits * head_dim;
    const size_t ml_floats = (size_t)batch * n_q_heads * splits * 2;
    if (acc_floats + ml_floats > kScratchFloats) return PYR_ERR_SCRATCH_LIMIT;
    // every slot the combine step reads is written by the split kernel of the
    // same call first, so nothing has to be cleared
    a.part_acc = base;
    a.part_ml = base + acc_floats;
  }
  if (pyr::launch_decode(a, static_cast<cudaStream_t>(stream)) != cudaSuccess) return PYR_ERR_CUDA;
  pyr::count_launches(splits > 1 ? 2 : 1);
  return PYR_OK;
}

extern "C" pyr_status_t pyr_decode_attn_noalloc_status(void* stream, int32_t* host_status) {
  if (!host_status) return PYR_ERR_NULL;
  float* base = nullptr;
  int* status_word = nullptr;
  pyr_status_t st = scratch_for_current_device(&base, &status_word);
  if (st != PYR_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int word = 0;
  const int zero = 0;
  if (cudaMemcpyAsync(&word, status_word, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return PYR_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return PYR_ERR_CUDA;
  if (word != 0) {     // report it once, then start clean
    if (cudaMemcpyAsync(status_word, &zero, sizeof(int), cudaMemcpyHostToDevice, s) != cudaSuccess) return PYR_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return PYR_ERR_CUDA;
  }
  *host_status = word;
  return word == 0 ? PYR_OK : PYR_ERR_TIMEOUT;
}
