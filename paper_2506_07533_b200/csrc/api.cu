// C ABI of the library: argument validation and dispatch to the kernel launchers.
#include <atomic>
#include <vector>

#include "common.cuh"

namespace {

thread_local int g_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return MOQAE_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int n_groups(const moqae_config* c) { return (c->n_layers + c->rs_group - 1) / c->rs_group; }

int check_config(const moqae_config* c) {
  if (!c) return MOQAE_ERR_INVALID_ARG;
  if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->batch < 1 || c->rs_group < 1 ||
      c->max_tokens < 0 || c->tail_capacity < 0 || c->chunk < 1)
    return MOQAE_ERR_INVALID_ARG;
  if (c->rf_first_chunk != 0 && c->rf_first_chunk != 1) return MOQAE_ERR_INVALID_ARG;
  if (c->head_dim != moqae::kHeadDim || c->group != moqae::kGroup || c->n_experts != MOQAE_N_EXPERTS)
    return MOQAE_ERR_UNSUPPORTED;
  for (int w = 0; w < 4; ++w)
    if (c->expert_bits[w] != moqae::bits_of_expert(w)) return MOQAE_ERR_UNSUPPORTED;
  if (c->chunk % moqae::kTileTokens != 0 && c->chunk != 8 && c->chunk != 16) return MOQAE_ERR_UNSUPPORTED;
  if (c->dtype != MOQAE_DTYPE_FP16 && c->dtype != MOQAE_DTYPE_BF16) return MOQAE_ERR_UNSUPPORTED;
  if (c->n_q_heads % c->n_kv_heads != 0) return MOQAE_ERR_INVALID_ARG;
  if (c->n_q_heads / c->n_kv_heads > moqae::kMaxQueryGroup) return MOQAE_ERR_UNSUPPORTED;
  if (c->d_in < 32 || c->d_in % 32 != 0) return MOQAE_ERR_UNSUPPORTED;
  if (c->per_head_routing != 0 && c->per_head_routing != 1) return MOQAE_ERR_INVALID_ARG;
  if (c->per_head_routing && c->d_in != moqae::kHeadDim) return MOQAE_ERR_UNSUPPORTED;
  return MOQAE_OK;
}

moqae::Dims dims_of(const moqae_config* c) {
  moqae::Dims d;
  d.n_layers = c->n_layers;
  d.n_q_heads = c->n_q_heads;
  d.n_kv_heads = c->n_kv_heads;
  d.chunk = c->chunk;
  d.dtype = c->dtype;
  d.rs_group = c->rs_group;
  d.rf_first_chunk = c->rf_first_chunk;
  d.d_in = c->d_in;
  d.max_chunks = c->max_tokens / c->chunk;
  d.tail_capacity = c->tail_capacity;
  d.batch = c->batch;
  d.per_head = c->per_head_routing ? 1 : 0;
  d.n_tseq = d.per_head ? c->batch * c->n_kv_heads : c->batch;
  return d;
}

int check_cache(const moqae_cache* k, moqae::CacheView* v) {
  if (!k) return MOQAE_ERR_INVALID_ARG;
  for (int w = 0; w < 4; ++w) {
    if (k->capacity[w] < 0) return MOQAE_ERR_INVALID_ARG;
    if (k->capacity[w] > 0 && !k->pool[w]) return MOQAE_ERR_INVALID_ARG;
    if (!aligned16(k->pool[w])) return MOQAE_ERR_MISALIGNED;
    v->pool[w] = static_cast<uint8_t*>(k->pool[w]);
    v->capacity[w] = k->capacity[w];
  }
  if (!k->map || !k->slot || !k->count || !k->votes || !k->tail_len || !k->status) return MOQAE_ERR_INVALID_ARG;
  if (!aligned16(k->slot) || !aligned16(k->count) || !aligned16(k->votes) || !aligned16(k->tail_k) ||
      !aligned16(k->tail_v) || !aligned16(k->status))
    return MOQAE_ERR_MISALIGNED;
  v->map = k->map;
  v->slot = k->slot;
  v->count = k->count;
  v->votes = k->votes;
  v->tail_k = static_cast<uint16_t*>(k->tail_k);
  v->tail_v = static_cast<uint16_t*>(k->tail_v);
  v->tail_len = k->tail_len;
  v->status = k->status;
  return MOQAE_OK;
}

}  // namespace

namespace moqae {
void record_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int>(e); }

int sm_count_of_current_device() {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cached[kMaxDevices];          // zero = not looked up yet
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  int v = cached[dev].load(std::memory_order_relaxed);
  if (v == 0) {
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    cached[dev].store(v, std::memory_order_relaxed);
  }
  return v;
}
}  // namespace moqae

#pragma GCC visibility push(default)
extern "C" {

int moqae_version(void) { return 200; }

int moqae_last_cuda_error(void) { return g_last_cuda_error; }

const char* moqae_error_string(int code) {
  switch (code) {
    case MOQAE_OK: return "ok";
    case MOQAE_ERR_INVALID_ARG: return "invalid argument";
    case MOQAE_ERR_UNSUPPORTED: return "unsupported configuration";
    case MOQAE_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case MOQAE_ERR_POOL_FULL: return "pool or tail capacity exceeded";
    case MOQAE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MOQAE_ERR_CUDA: return "CUDA runtime error (see moqae_last_cuda_error)";
    case MOQAE_ERR_TIMEOUT: return "bounded device wait expired";
    case MOQAE_ERR_CORRUPT_TABLE: return "chunk index table breaks the slot rules";
    default: return "unknown error";
  }
}

int moqae_cache_bytes(const moqae_config* cfg, const int64_t capacity[4], int64_t out_bytes[MOQAE_N_CACHE_BUFFERS]) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  if (!capacity || !out_bytes) return MOQAE_ERR_INVALID_ARG;
  const int64_t lbh = static_cast<int64_t>(cfg->n_layers) * cfg->batch * cfg->n_kv_heads;
  const int64_t tpc = moqae::tiles_per_chunk_of(cfg->chunk);
  for (int w = 0; w < 4; ++w) {
    if (capacity[w] < 0) return MOQAE_ERR_INVALID_ARG;
    out_bytes[w] = lbh * capacity[w] * tpc * moqae::tile_bytes_of_expert(w);
  }
  const int64_t rows = cfg->per_head_routing ? static_cast<int64_t>(cfg->batch) * cfg->n_kv_heads : cfg->batch;
  const int64_t tbl = static_cast<int64_t>(n_groups(cfg)) * rows * (cfg->max_tokens / cfg->chunk);
  out_bytes[4] = tbl;                                   // map, uint8
  out_bytes[5] = tbl * 4;                               // slot
  out_bytes[6] = static_cast<int64_t>(n_groups(cfg)) * rows * 4 * 4;         // count
  out_bytes[7] = tbl * 16;                              // votes
  out_bytes[8] = lbh * cfg->tail_capacity * moqae::kHeadDim * 2;
  out_bytes[9] = out_bytes[8];
  out_bytes[10] = static_cast<int64_t>(cfg->n_layers) * cfg->batch * 4;
  out_bytes[11] = 16;
  return MOQAE_OK;
}

int moqae_cache_bind(const moqae_config* cfg, const int64_t capacity[4], void* const buffers[MOQAE_N_CACHE_BUFFERS],
                     moqae_cache* out) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  if (!capacity || !buffers || !out) return MOQAE_ERR_INVALID_ARG;
  for (int i = 0; i < MOQAE_N_CACHE_BUFFERS; ++i)
    if (!aligned16(buffers[i])) return MOQAE_ERR_MISALIGNED;
  for (int w = 0; w < 4; ++w) {
    out->pool[w] = buffers[w];
    out->capacity[w] = capacity[w];
  }
  out->map = static_cast<uint8_t*>(buffers[4]);
  out->slot = static_cast<int32_t*>(buffers[5]);
  out->count = static_cast<int32_t*>(buffers[6]);
  out->votes = static_cast<int32_t*>(buffers[7]);
  out->tail_k = buffers[8];
  out->tail_v = buffers[9];
  out->tail_len = static_cast<int32_t*>(buffers[10]);
  out->status = static_cast<int32_t*>(buffers[11]);
  moqae::CacheView v;
  return check_cache(out, &v);
}

int moqae_route(const moqae_config* cfg, const void* hidden, int32_t T, const void* W1, const void* W2,
                const float* W3, const float* bias, int32_t layer_group, const moqae_cache* cache,
                int32_t* votes_out, void* stream) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (!hidden || !W1 || T < 0 || T > cfg->max_tokens) return MOQAE_ERR_INVALID_ARG;
  if ((W2 == nullptr) != (W3 == nullptr)) return MOQAE_ERR_INVALID_ARG;
  if (layer_group < 0 || layer_group >= n_groups(cfg)) return MOQAE_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(W1) || !aligned16(W2) || !aligned16(W3) || !aligned16(bias) ||
      !aligned16(votes_out))
    return MOQAE_ERR_MISALIGNED;
  cudaError_t e = moqae::launch_route(dims_of(cfg), cv, hidden, T, W1, W2, W3, bias, layer_group, votes_out,
                                      static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOQAE_OK : cuda_fail(e);
}

int moqae_quantize_kv(const moqae_config* cfg, const void* K, const void* V, int32_t T, int32_t layer,
                      const uint8_t* forced_map, const moqae_cache* cache, void* stream) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (T < 0 || T > cfg->max_tokens || layer < 0 || layer >= cfg->n_layers) return MOQAE_ERR_INVALID_ARG;
  if (T > 0 && (!K || !V)) return MOQAE_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V)) return MOQAE_ERR_MISALIGNED;
  if (T % cfg->chunk > cfg->tail_capacity) return MOQAE_ERR_POOL_FULL;
  if (cfg->tail_capacity > 0 && (!cache->tail_k || !cache->tail_v)) return MOQAE_ERR_INVALID_ARG;
  const moqae::Dims dm = dims_of(cfg);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (forced_map) {
    cudaError_t e = moqae::launch_finalize_map(dm, cv, layer / cfg->rs_group, T / cfg->chunk, forced_map, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  cudaError_t e = moqae::launch_quantize(dm, cv, K, V, T, layer, st);
  return e == cudaSuccess ? MOQAE_OK : cuda_fail(e);
}

int moqae_project_quantize_kv(const moqae_config* cfg, const void* hidden, const void* Wk, const void* Wv, int32_t T,
                              int32_t layer, const uint8_t* forced_map, const moqae_cache* cache, void* k_rounded,
                              void* v_rounded, void* stream) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (T < 0 || T > cfg->max_tokens || layer < 0 || layer >= cfg->n_layers) return MOQAE_ERR_INVALID_ARG;
  if (T > 0 && (!hidden || !Wk || !Wv)) return MOQAE_ERR_INVALID_ARG;
  if ((k_rounded == nullptr) != (v_rounded == nullptr)) return MOQAE_ERR_INVALID_ARG;
  if (cfg->d_in % 64 != 0 || cfg->chunk < moqae::kTileTokens || cfg->per_head_routing) return MOQAE_ERR_UNSUPPORTED;
  if (!aligned16(hidden) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(k_rounded) || !aligned16(v_rounded))
    return MOQAE_ERR_MISALIGNED;
  if (T % cfg->chunk > cfg->tail_capacity) return MOQAE_ERR_POOL_FULL;
  if (cfg->tail_capacity > 0 && (!cache->tail_k || !cache->tail_v)) return MOQAE_ERR_INVALID_ARG;
  const moqae::Dims dm = dims_of(cfg);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (forced_map) {
    cudaError_t e = moqae::launch_finalize_map(dm, cv, layer / cfg->rs_group, T / cfg->chunk, forced_map, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  cudaError_t e = moqae::launch_project_quantize(dm, cv, hidden, Wk, Wv, T, layer, k_rounded, v_rounded, st);
  return e == cudaSuccess ? MOQAE_OK : cuda_fail(e);
}

int moqae_append_kv(const moqae_config* cfg, const void* k_new, const void* v_new, int32_t layer,
                    const moqae_cache* cache, void* stream) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (!k_new || !v_new || layer < 0 || layer >= cfg->n_layers) return MOQAE_ERR_INVALID_ARG;
  if (cfg->tail_capacity < 1 || !cache->tail_k || !cache->tail_v) return MOQAE_ERR_POOL_FULL;
  if (!aligned16(k_new) || !aligned16(v_new)) return MOQAE_ERR_MISALIGNED;
  cudaError_t e = moqae::launch_append(dims_of(cfg), cv, k_new, v_new, layer, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOQAE_OK : cuda_fail(e);
}

int moqae_flush_tail(const moqae_config* cfg, const void* hidden_tail, const void* W1, const void* W2,
                     const float* W3, const float* bias, int32_t layer_group, const moqae_cache* cache,
                     void* stream) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (!hidden_tail || !W1) return MOQAE_ERR_INVALID_ARG;
  if ((W2 == nullptr) != (W3 == nullptr)) return MOQAE_ERR_INVALID_ARG;
  if (layer_group < 0 || layer_group >= n_groups(cfg)) return MOQAE_ERR_INVALID_ARG;
  if (cfg->tail_capacity < cfg->chunk || !cache->tail_k || !cache->tail_v) return MOQAE_ERR_POOL_FULL;
  if (cfg->per_head_routing) return MOQAE_ERR_UNSUPPORTED;               // the flush keeps one table row per sequence
  if (!aligned16(hidden_tail) || !aligned16(W1) || !aligned16(W2) || !aligned16(W3) || !aligned16(bias))
    return MOQAE_ERR_MISALIGNED;
  const moqae::Dims dm = dims_of(cfg);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = moqae::launch_flush_route(dm, cv, hidden_tail, W1, W2, W3, bias, layer_group, st);
  const int l0 = layer_group * cfg->rs_group;
  for (int l = l0; e == cudaSuccess && l < l0 + cfg->rs_group && l < cfg->n_layers; ++l)
    e = moqae::launch_flush_quantize(dm, cv, l, st);
  if (e == cudaSuccess) e = moqae::launch_flush_reset(dm, cv, layer_group, st);
  return e == cudaSuccess ? MOQAE_OK : cuda_fail(e);
}

int moqae_decode_attn_workspace(const moqae_config* cfg, int64_t* out_bytes) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  if (!out_bytes) return MOQAE_ERR_INVALID_ARG;
  const moqae::Dims dm = dims_of(cfg);
  *out_bytes = moqae::decode_workspace_bytes(dm, moqae::decode_num_splits(dm));
  return MOQAE_OK;
}

int moqae_decode_attn(const moqae_config* cfg, const void* q, int32_t layer, const moqae_cache* cache,
                      float* out, float scale, void* workspace, int64_t workspace_bytes, void* stream) {
  return moqae_decode_attn_ex(cfg, q, layer, cache, out, scale, workspace, workspace_bytes, 0, stream);
}

int moqae_decode_attn_ex(const moqae_config* cfg, const void* q, int32_t layer, const moqae_cache* cache,
                         float* out, float scale, void* workspace, int64_t workspace_bytes, int32_t flags,
                         void* stream) {
  return moqae_decode_attn_step(cfg, q, nullptr, nullptr, layer, cache, out, scale, workspace, workspace_bytes, flags, stream);
}

int moqae_decode_attn_step(const moqae_config* cfg, const void* q, const void* k_new, const void* v_new, int32_t layer,
                           const moqae_cache* cache, float* out, float scale, void* workspace, int64_t workspace_bytes,
                           int32_t flags, void* stream) {
  if (flags & ~MOQAE_DECODE_OVERLAP_PREVIOUS) return MOQAE_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return MOQAE_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return MOQAE_ERR_MISALIGNED;
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (!q || !out || !workspace || layer < 0 || layer >= cfg->n_layers) return MOQAE_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return MOQAE_ERR_MISALIGNED;
  const moqae::Dims dm = dims_of(cfg);
  const int s = moqae::decode_num_splits(dm);
  const int64_t need = moqae::decode_workspace_bytes(dm, s);
  if (workspace_bytes < need) return MOQAE_ERR_WORKSPACE_TOO_SMALL;
  if (!(scale > 0.0f)) scale = 0.08838834764831845f;   // 1/sqrt(128)
  cudaError_t e = moqae::launch_decode(dm, cv, q, layer, out, scale, static_cast<float*>(workspace), s,
                                       (flags & MOQAE_DECODE_OVERLAP_PREVIOUS) != 0, k_new, v_new,
                                       static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOQAE_OK : cuda_fail(e);
}

int moqae_prefill_attn_workspace(const moqae_config* cfg, int32_t T, int64_t* bytes) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  if (!bytes || T < 0 || T > cfg->max_tokens) return MOQAE_ERR_INVALID_ARG;
  *bytes = moqae::prefill_workspace_bytes(dims_of(cfg), T);
  return MOQAE_OK;
}

int moqae_prefill_attn(const moqae_config* cfg, const void* q, int32_t T, int32_t layer, const moqae_cache* cache,
                       float* out, float scale, void* workspace, int64_t workspace_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (T < 0 || T > cfg->max_tokens || layer < 0 || layer >= cfg->n_layers) return MOQAE_ERR_INVALID_ARG;
  if (cfg->chunk < moqae::kTileTokens) return MOQAE_ERR_UNSUPPORTED;     // walks the cache in whole 32-token tiles
  if (cfg->per_head_routing) return MOQAE_ERR_UNSUPPORTED;               // reads one map per sequence
  if (T > 0 && (!q || !out)) return MOQAE_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return MOQAE_ERR_MISALIGNED;
  if (workspace && workspace_bytes < moqae::prefill_workspace_bytes(dims_of(cfg), T)) return MOQAE_ERR_WORKSPACE_TOO_SMALL;
  if (!(scale > 0.0f)) scale = 0.08838834764831845f;   // 1/sqrt(128)
  cudaError_t e = moqae::launch_prefill_attn(dims_of(cfg), cv, q, T, layer, scale, out, workspace, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MOQAE_OK : cuda_fail(e);
}

int moqae_validate_tables_host(const uint8_t* map, const int32_t* slot, const int32_t* count, int32_t rows,
                               int32_t max_chunks, int32_t n_chunks, const int64_t capacity[4], int32_t* bad_row,
                               int32_t* bad_chunk) {
  if (!map || !slot || !count || !capacity || rows < 0 || n_chunks < 0 || n_chunks > max_chunks) return MOQAE_ERR_INVALID_ARG;
  auto fail = [&](int r, int c) {
    if (bad_row) *bad_row = r;
    if (bad_chunk) *bad_chunk = c;
    return MOQAE_ERR_CORRUPT_TABLE;
  };
  for (int r = 0; r < rows; ++r) {
    int64_t seen[4] = {0, 0, 0, 0};
    for (int c = 0; c < n_chunks; ++c) {
      const int w = map[static_cast<int64_t>(r) * max_chunks + c];
      if (w > 3) return fail(r, c);
      const int32_t s = slot[static_cast<int64_t>(r) * max_chunks + c];
      if (s != seen[w] || s >= capacity[w]) return fail(r, c);
      seen[w]++;
    }
    for (int w = 0; w < 4; ++w)
      if (count[4 * r + w] != seen[w]) return fail(r, -1);
  }
  return MOQAE_OK;
}

int moqae_validate_tables(const moqae_config* cfg, const moqae_cache* cache, int32_t T, int32_t layer_group,
                          void* stream, int32_t* bad_row, int32_t* bad_chunk) {
  int rc = check_config(cfg);
  if (rc != MOQAE_OK) return rc;
  moqae::CacheView cv;
  rc = check_cache(cache, &cv);
  if (rc != MOQAE_OK) return rc;
  if (T < 0 || T > cfg->max_tokens || layer_group < 0 || layer_group >= n_groups(cfg)) return MOQAE_ERR_INVALID_ARG;
  const moqae::Dims dm = dims_of(cfg);
  const int64_t rows = dm.n_tseq, mc = dm.max_chunks;
  std::vector<uint8_t> map(static_cast<size_t>(rows * mc));
  std::vector<int32_t> slot(static_cast<size_t>(rows * mc)), count(static_cast<size_t>(rows * 4));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(map.data(), cv.map + layer_group * rows * mc, map.size(), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(slot.data(), cv.slot + layer_group * rows * mc, slot.size() * 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(count.data(), cv.count + layer_group * rows * 4, count.size() * 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e);
  return moqae_validate_tables_host(map.data(), slot.data(), count.data(), static_cast<int32_t>(rows), static_cast<int32_t>(mc),
                                    T / cfg->chunk, cache->capacity, bad_row, bad_chunk);
}

int moqae_poll_status(const moqae_cache* cache, void* stream, int32_t* out_status) {
  if (!cache || !cache->status || !out_status) return MOQAE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t h[4] = {0, 0, 0, 0};
  cudaError_t e = cudaMemcpyAsync(h, cache->status, sizeof(h), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e);
  *out_status = h[0];
  return MOQAE_OK;
}

}  // extern "C"
#pragma GCC visibility pop
