// Split-K decode attention over the mixed-precision cache (flash-decoding style): launch logic.
//
// Softmax attention does not depend on the order of the keys, so a CTA does not walk the
// chunks in sequence order: for its (sequence, kv head) it walks pool by pool - all 2-bit
// tiles, then the 4-bit, 8-bit and 16-bit ones, then (last split only) the 16-bit tail.
// Each (sequence, kv head) is cut into n_splits pieces, every piece taking the same share
// of every pool, so all CTAs stream the same bytes AND the same mix of widths.
// Each CTA writes, per query head of the group, a partial (max, sum, 128 weighted values);
// the CTA that arrives last for a (sequence, kv head) merges the partials with the
// log-sum-exp rule and writes the output (decode_mma.cu).
#include "common.cuh"

namespace moqae {

int decode_num_splits(const Dims& dm) {
  const int sms = sm_count_of_current_device();
  // one full wave: every CTA gets the same number of bytes, so a partial second wave would
  // cost a whole extra pass
  const int pairs = dm.batch * dm.n_kv_heads;
  int s = (sms * decode_mma_ctas_per_sm()) / pairs;
  if (s < 1) s = 1;
  if (s > kMaxSplits) s = kMaxSplits;
  return s;
}

// workspace: ws_o [batch][n_q_heads][n_splits][128] floats, ws_ml [batch][n_q_heads][n_splits][2]
// floats, then one arrival counter per (sequence, kv head)
long long decode_workspace_bytes(const Dims& dm, int n_splits) {
  const long long rows = static_cast<long long>(dm.batch) * dm.n_q_heads * n_splits;
  const long long bytes = rows * (kHeadDim + 2) * 4 + static_cast<long long>(dm.batch) * dm.n_kv_heads * 4;
  return (bytes + 15) / 16 * 16;
}

void decode_counter_region(const moqae_config* cfg, long long* offset, long long* bytes) {
  Dims dm{};
  dm.batch = cfg->batch;
  dm.n_q_heads = cfg->n_q_heads;
  dm.n_kv_heads = cfg->n_kv_heads;
  const long long rows = static_cast<long long>(dm.batch) * dm.n_q_heads * decode_num_splits(dm);
  *offset = rows * (kHeadDim + 2) * 4;
  *bytes = static_cast<long long>(dm.batch) * dm.n_kv_heads * 4;
}

cudaError_t launch_decode(const Dims& dm, const CacheView& cv, const void* q, int layer, float* out,
                          float scale, float* workspace, int n_splits, bool overlap_previous, const void* k_new,
                          const void* v_new, cudaStream_t st) {
  const long long rows = static_cast<long long>(dm.batch) * dm.n_q_heads * n_splits;
  float* ws_o = workspace;
  float* ws_ml = workspace + rows * kHeadDim;
  int* arrived = reinterpret_cast<int*>(ws_ml + rows * 2);
  // the counters are zero on entry (the caller zeroes a new workspace once) and the kernel
  // leaves them zero: the last arrival of every (sequence, kv head) wraps its counter around
  return launch_decode_mma(dm, cv, q, layer, scale, ws_o, ws_ml, arrived, out, n_splits, overlap_previous, k_new, v_new, st);
}

}  // namespace moqae
