// Shared declarations of the MoQAE CUDA library (sm_100a).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moqae.h"

namespace moqae {

constexpr int kHeadDim = 128;
constexpr int kGroup = 32;
constexpr int kTileTokens = 32;
constexpr int kMetaBytes = 1024;
constexpr int kRawTileBytes = 16384;
constexpr int kMaxQueryGroup = 8;
constexpr int kMaxSplits = 64;

__host__ __device__ constexpr int bits_of_expert(int w) { return 2 << w; }   // 2,4,8,16
__host__ __device__ constexpr int tile_bytes_of_expert(int w) {
  return w == 3 ? kRawTileBytes : kMetaBytes + 1024 * (2 << w);
}

// A chunk of 32 j tokens is j tiles; a chunk of 8 or 16 tokens is one tile whose first `chunk`
// token positions hold tokens (the rest is padding: codes 0, never attended).
__host__ __device__ constexpr int tiles_per_chunk_of(int chunk) { return chunk >= kTileTokens ? chunk / kTileTokens : 1; }
__host__ __device__ constexpr int tile_tokens_of(int chunk) { return chunk >= kTileTokens ? kTileTokens : chunk; }

// Everything a kernel needs to find its way around a cache (passed by value).
struct CacheView {
  uint8_t* pool[4];
  long long capacity[4];
  uint8_t* map;
  int32_t* slot;
  int32_t* count;
  int32_t* votes;
  uint16_t* tail_k;
  uint16_t* tail_v;
  int32_t* tail_len;
  int32_t* status;
};

struct Dims {
  int n_layers, n_q_heads, n_kv_heads, chunk, dtype, rs_group, rf_first_chunk, d_in;
  int max_chunks, tail_capacity, batch;
  int per_head;        // 1: one table row per (sequence, kv head) instead of one per sequence
  int n_tseq;          // table rows per routing-sharing group: batch, or batch * n_kv_heads
};

// table row of (sequence b, kv head h)
__host__ __device__ __forceinline__ int table_row(const Dims& dm, int b, int h) {
  return dm.per_head ? b * dm.n_kv_heads + h : b;
}

__device__ __forceinline__ void set_status(int32_t* status, int code, int d0, int d1) {
  if (atomicCAS(status, 0, code) == 0) {
    status[1] = d0;
    status[2] = d1;
  }
}

__device__ __forceinline__ float load16_as_float(uint16_t u, int dtype) {
  return dtype == MOQAE_DTYPE_FP16 ? __half2float(__ushort_as_half(u))
                                   : __uint_as_float(static_cast<uint32_t>(u) << 16);
}

// Address of slot `slot` of (layer, b, h) in pool w.
__device__ __forceinline__ uint8_t* slot_ptr(const CacheView& cv, const Dims& dm, int w, int layer,
                                             int b, int h, long long slot) {
  const long long slot_bytes = static_cast<long long>(tiles_per_chunk_of(dm.chunk)) * tile_bytes_of_expert(w);
  const long long idx = ((static_cast<long long>(layer) * dm.batch + b) * dm.n_kv_heads + h) *
                            cv.capacity[w] + slot;
  return cv.pool[w] + idx * slot_bytes;
}

// Number of SMs of the device that is current on the calling thread (looked up once per device).
int sm_count_of_current_device();

// Remember `e` as the code moqae_last_cuda_error() reports on this thread.
void record_cuda_error(cudaError_t e);

// Launchers implemented in the .cu files (host side, return cudaError_t).
cudaError_t launch_route(const Dims& dm, const CacheView& cv, const void* hidden, int T, const void* W1,
                         const void* W2, const float* W3, const float* bias, int group,
                         int32_t* votes_out, cudaStream_t st);
cudaError_t launch_flush_route(const Dims& dm, const CacheView& cv, const void* hidden_tail, const void* W1,
                               const void* W2, const float* W3, const float* bias, int group, cudaStream_t st);
cudaError_t launch_flush_quantize(const Dims& dm, const CacheView& cv, int layer, cudaStream_t st);
cudaError_t launch_flush_reset(const Dims& dm, const CacheView& cv, int group, cudaStream_t st);
cudaError_t launch_finalize_map(const Dims& dm, const CacheView& cv, int group, int n_chunks,
                                const uint8_t* forced_map, cudaStream_t st);
cudaError_t launch_quantize(const Dims& dm, const CacheView& cv, const void* K, const void* V, int T,
                            int layer, cudaStream_t st);
cudaError_t launch_append(const Dims& dm, const CacheView& cv, const void* k_new, const void* v_new,
                          int layer, cudaStream_t st);
cudaError_t launch_project_quantize(const Dims& dm, const CacheView& cv, const void* hidden, const void* Wk, const void* Wv,
                                    int T, int layer, void* dbg_k, void* dbg_v, cudaStream_t st);
int decode_num_splits(const Dims& dm);
int decode_mma_ctas_per_sm();
cudaError_t launch_prefill_attn(const Dims& dm, const CacheView& cv, const void* q, int T, int layer, float scale,
                                float* out, void* workspace, cudaStream_t st);
long long prefill_workspace_bytes(const Dims& dm, int T);
long long decode_workspace_bytes(const Dims& dm, int n_splits);
// byte offset and length of the arrival counters inside a decode workspace for `cfg`
void decode_counter_region(const moqae_config* cfg, long long* offset, long long* bytes);
cudaError_t launch_decode_mma(const Dims& dm, const CacheView& cv, const void* q, int layer, float scale,
                              float* ws_o, float* ws_ml, int* arrived, float* out, int n_splits, bool overlap_previous,
                              const void* k_new, const void* v_new, cudaStream_t st);
cudaError_t launch_decode(const Dims& dm, const CacheView& cv, const void* q, int layer, float* out,
                          float scale, float* workspace, int n_splits, bool overlap_previous, const void* k_new,
                          const void* v_new, cudaStream_t st);

}  // namespace moqae
