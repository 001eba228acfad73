// Split-K decode attention over the mixed-precision cache (flash-decoding style): launch
// logic and the split combine.
//
// Softmax attention does not depend on the order of the keys, so a CTA does not walk the
// chunks in sequence order: for its (sequence, kv head) it walks pool by pool - all 2-bit
// tiles, then the 4-bit, 8-bit and 16-bit ones, then (last split only) the 16-bit tail.
// Each (sequence, kv head) is cut into n_splits pieces, every piece taking the same share
// of every pool, so all CTAs stream the same bytes AND the same mix of widths.
// Each CTA writes, per query head of the group, a partial (max, sum, 128 weighted values)
// (decode_mma.cu); decode_combine_kernel merges the partials with the log-sum-exp rule.
#include "common.cuh"

namespace moqae {

namespace {

// out[b][hq][c] = sum_s o_s e^{m_s - m*} / sum_s l_s e^{m_s - m*}
__global__ void __launch_bounds__(kHeadDim)
decode_combine_kernel(const float* __restrict__ ws_o, const float* __restrict__ ws_ml, float* __restrict__ out,
                      int n_splits) {
  const long long row0 = static_cast<long long>(blockIdx.x) * n_splits;
  const int c = threadIdx.x;
  float m = -INFINITY;
  for (int s = 0; s < n_splits; ++s) m = fmaxf(m, ws_ml[(row0 + s) * 2]);
  float l = 0.0f, o = 0.0f;
  for (int s = 0; s < n_splits; ++s) {
    const float ms = ws_ml[(row0 + s) * 2];
    const float f = (ms == -INFINITY) ? 0.0f : __expf(ms - m);
    l += ws_ml[(row0 + s) * 2 + 1] * f;
    o += ws_o[(row0 + s) * kHeadDim + c] * f;
  }
  out[static_cast<long long>(blockIdx.x) * kHeadDim + c] = l > 0.0f ? o / l : 0.0f;
}

}  // namespace

int decode_num_splits(const Dims& dm) {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, v = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    sms = v > 0 ? v : 148;
  }
  // one full wave: every CTA gets the same number of bytes, so a partial second wave would
  // cost a whole extra pass
  const int pairs = dm.batch * dm.n_kv_heads;
  int s = (sms * decode_mma_ctas_per_sm()) / pairs;
  if (s < 1) s = 1;
  if (s > kMaxSplits) s = kMaxSplits;
  return s;
}

// workspace: ws_o [batch][n_q_heads][n_splits][128] then ws_ml [batch][n_q_heads][n_splits][2]
cudaError_t launch_decode(const Dims& dm, const CacheView& cv, const void* q, int layer, float* out,
                          float scale, float* workspace, int n_splits, cudaStream_t st) {
  const long long rows = static_cast<long long>(dm.batch) * dm.n_q_heads * n_splits;
  float* ws_o = workspace;
  float* ws_ml = workspace + rows * kHeadDim;
  cudaError_t e = launch_decode_mma(dm, cv, q, layer, scale, ws_o, ws_ml, n_splits, st);
  if (e != cudaSuccess) return e;
  decode_combine_kernel<<<dm.batch * dm.n_q_heads, kHeadDim, 0, st>>>(ws_o, ws_ml, out, n_splits);
  return cudaGetLastError();
}

}  // namespace moqae
