// Split-K decode attention over the mixed-precision cache (flash-decoding style).
//
// Softmax attention does not depend on the order of the keys, so a CTA does not walk the
// chunks in sequence order: for its (sequence, kv head) it walks pool by pool - all 2-bit
// tiles, then the 4-bit, 8-bit and 16-bit ones, then (last split only) the 16-bit tail.
// Each (sequence, kv head) is cut into n_splits pieces of equal COST, a tile costing its
// size in KiB (3, 5, 9, 16), so every CTA streams about the same number of bytes.
// Each CTA writes, per query head of the group, a partial (max, sum, 128 weighted values);
// decode_combine_kernel merges the partials with the log-sum-exp rule.
#include <cstdlib>

#include "common.cuh"

namespace moqae {

namespace {

constexpr int kDecWarps = 4;

struct SplitRange {
  int lo[4], hi[4];   // tile range per width inside the (layer, b, h, w) stream
};

// Tiles of width w whose cost-axis start lies in [lo_cost, hi_cost).
__device__ __forceinline__ SplitRange split_range(const int32_t* cnt_in, const long long* capacity,
                                                  int tiles_per_chunk, int split, int n_splits) {
  int cnt[4];   // never walk past a pool's end, whatever the table says
#pragma unroll
  for (int w = 0; w < 4; ++w) cnt[w] = static_cast<int>(min(static_cast<long long>(max(cnt_in[w], 0)), capacity[w]));
  long long base[5];
  base[0] = 0;
#pragma unroll
  for (int w = 0; w < 4; ++w)
    base[w + 1] = base[w] + static_cast<long long>(cnt[w]) * tiles_per_chunk * tile_cost_of_expert(w);
  const long long total = base[4];
  const long long lo_c = total * split / n_splits, hi_c = total * (split + 1) / n_splits;
  SplitRange r;
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const long long cost = tile_cost_of_expert(w);
    const long long n = static_cast<long long>(cnt[w]) * tiles_per_chunk;
    long long a = lo_c - base[w], b = hi_c - base[w];
    a = a <= 0 ? 0 : (a + cost - 1) / cost;
    b = b <= 0 ? 0 : (b + cost - 1) / cost;
    r.lo[w] = static_cast<int>(a < n ? a : n);
    r.hi[w] = static_cast<int>(b < n ? b : n);
  }
  return r;
}

struct WarpState {
  float m[kMaxQueryGroup];
  float l[kMaxQueryGroup];
  float acc[kMaxQueryGroup][4];   // channels 4*lane .. 4*lane+3
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Fold the scores of 32 tokens (one per lane; -inf = masked) into the running state and
// return this lane's softmax numerators in p[].
template <int G>
__device__ __forceinline__ void online_update(WarpState& st, const float s[G], float p[G]) {
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const float mt = warp_max(s[g]);
    const float mnew = fmaxf(st.m[g], mt);
    const float corr = (mnew == -INFINITY) ? 1.0f : __expf(st.m[g] - mnew);
    p[g] = (s[g] == -INFINITY) ? 0.0f : __expf(s[g] - mnew);
    st.l[g] = st.l[g] * corr + warp_sum(p[g]);
#pragma unroll
    for (int k = 0; k < 4; ++k) st.acc[g][k] *= corr;
    st.m[g] = mnew;
  }
}

// ---- quantised tile: lane = token for the scores, lane = 4 channels for the values
template <int BITS, int G>
__device__ void process_quant_tile(const uint8_t* __restrict__ tile, const float* __restrict__ qs /* smem [G][128], pre-scaled */,
                                   WarpState& st, int lane) {
  constexpr int n = 32 / BITS;
  constexpr uint32_t mask = (1u << BITS) - 1u;
  const __half* ks = reinterpret_cast<const __half*>(tile);
  const __half* kz = reinterpret_cast<const __half*>(tile + 256);
  const uint8_t* krow = tile + kMetaBytes + lane * 16 * BITS;
  float s[G];
#pragma unroll
  for (int g = 0; g < G; ++g) s[g] = 0.0f;
  for (int j = 0; j < 4 * BITS; ++j) {      // logical words of this token's row
    int unit = j >> 2;
    if (BITS == 8) unit ^= (lane & 7);
    const uint32_t wv = *reinterpret_cast<const uint32_t*>(krow + unit * 16 + (j & 3) * 4);
#pragma unroll
    for (int i = 0; i < n; ++i) {
      const int c = j * n + i;
      const float code = static_cast<float>((wv >> (BITS * (i >> 1) + 16 * (i & 1))) & mask);
      const float kh = fmaf(code, __half2float(ks[c]), __half2float(kz[c]));
#pragma unroll
      for (int g = 0; g < G; ++g) s[g] = fmaf(qs[g * kHeadDim + c], kh, s[g]);
    }
  }
  float p[G];
  online_update<G>(st, s, p);
  // values: this lane accumulates channels 32*cg + 4*u + k, stored at positions 16*u + 4*cg + k
  const int cg = lane >> 3, u = lane & 7;
  const int p0 = 16 * u + 4 * cg;
  const int j = p0 / n, i0 = p0 % n;
  const __half* vs = reinterpret_cast<const __half*>(tile + 512) + cg * 32;
  const __half* vz = reinterpret_cast<const __half*>(tile + 768) + cg * 32;
  const uint8_t* vpay = tile + kMetaBytes + kTileTokens * 16 * BITS;
  for (int t = 0; t < kTileTokens; ++t) {
    int unit = j >> 2;
    if (BITS == 8) unit ^= (t & 7);
    const uint32_t wv = *reinterpret_cast<const uint32_t*>(vpay + t * 16 * BITS + unit * 16 + (j & 3) * 4);
    const float sc = __half2float(vs[t]), zr = __half2float(vz[t]);
    float v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k;
      v[k] = fmaf(static_cast<float>((wv >> (BITS * (i >> 1) + 16 * (i & 1))) & mask), sc, zr);
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float pt = __shfl_sync(0xffffffffu, p[g], t);
#pragma unroll
      for (int k = 0; k < 4; ++k) st.acc[g][k] = fmaf(pt, v[k], st.acc[g][k]);
    }
  }
}

// ---- 16-bit rows.  SWIZZLED: pool tiles (256-byte rows, units swizzled); otherwise tail rows.
template <int G, bool SWIZZLED>
__device__ void process_raw_rows(const uint16_t* __restrict__ Krows, const uint16_t* __restrict__ Vrows,
                                 int n_valid, int dtype, const float* __restrict__ qs, WarpState& st, int lane) {
  float s[G];
#pragma unroll
  for (int g = 0; g < G; ++g) s[g] = 0.0f;
  if (lane < n_valid) {
    const uint16_t* kr = Krows + lane * kHeadDim;
    for (int U = 0; U < 16; ++U) {
      const int up = SWIZZLED ? ((U & 8) | ((U ^ lane) & 7)) : U;
      const uint4 raw = *reinterpret_cast<const uint4*>(kr + up * 8);
      const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float kh = load16_as_float(static_cast<uint16_t>(w4[i >> 1] >> (16 * (i & 1))), dtype);
#pragma unroll
        for (int g = 0; g < G; ++g) s[g] = fmaf(qs[g * kHeadDim + U * 8 + i], kh, s[g]);
      }
    }
  } else {
#pragma unroll
    for (int g = 0; g < G; ++g) s[g] = -INFINITY;
  }
  float p[G];
  online_update<G>(st, s, p);
  const int U = lane >> 1;
  for (int t = 0; t < n_valid; ++t) {
    const int up = SWIZZLED ? ((U & 8) | ((U ^ t) & 7)) : U;
    const uint2 raw = *reinterpret_cast<const uint2*>(Vrows + t * kHeadDim + up * 8 + (lane & 1) * 4);
    float v[4];
    v[0] = load16_as_float(static_cast<uint16_t>(raw.x), dtype);
    v[1] = load16_as_float(static_cast<uint16_t>(raw.x >> 16), dtype);
    v[2] = load16_as_float(static_cast<uint16_t>(raw.y), dtype);
    v[3] = load16_as_float(static_cast<uint16_t>(raw.y >> 16), dtype);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float pt = __shfl_sync(0xffffffffu, p[g], t);
#pragma unroll
      for (int k = 0; k < 4; ++k) st.acc[g][k] = fmaf(pt, v[k], st.acc[g][k]);
    }
  }
}

// Partials: ws_o [batch][n_q_heads][n_splits][128], ws_ml [batch][n_q_heads][n_splits][2].
template <int G>
__global__ void __launch_bounds__(kDecWarps * 32)
decode_splitk_kernel(Dims dm, CacheView cv, const uint16_t* __restrict__ q, int layer, float scale,
                     float* __restrict__ ws_o, float* __restrict__ ws_ml, int n_splits) {
  __shared__ float qs[G * kHeadDim];
  __shared__ float red_o[kDecWarps][G][kHeadDim];
  __shared__ float red_ml[kDecWarps][G][2];
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < G * kHeadDim; i += blockDim.x) {
    const int g = i / kHeadDim, c = i % kHeadDim;
    qs[i] = load16_as_float(q[(static_cast<long long>(b) * dm.n_q_heads + h * G + g) * kHeadDim + c], dm.dtype) * scale;
  }
  __syncthreads();

  const int group = layer / dm.rs_group;
  const int32_t* cnt = cv.count + (static_cast<long long>(group) * dm.batch + b) * 4;
  const int tpc = dm.chunk / kTileTokens;
  const SplitRange rg = split_range(cnt, cv.capacity, tpc, split, n_splits);

  WarpState st;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    st.m[g] = -INFINITY;
    st.l[g] = 0.0f;
#pragma unroll
    for (int k = 0; k < 4; ++k) st.acc[g][k] = 0.0f;
  }

#pragma unroll
  for (int w = 0; w < 4; ++w) {
    // slots of one (layer, b, h) are contiguous, and tiles inside a slot too: one flat stream
    const uint8_t* stream = slot_ptr(cv, dm, w, layer, b, h, 0);
    for (int t = rg.lo[w] + warp; t < rg.hi[w]; t += kDecWarps) {
      const uint8_t* tile = stream + static_cast<long long>(t) * tile_bytes_of_expert(w);
      if (w == 0) process_quant_tile<2, G>(tile, qs, st, lane);
      else if (w == 1) process_quant_tile<4, G>(tile, qs, st, lane);
      else if (w == 2) process_quant_tile<8, G>(tile, qs, st, lane);
      else process_raw_rows<G, true>(reinterpret_cast<const uint16_t*>(tile),
                                     reinterpret_cast<const uint16_t*>(tile + 8192), 32, dm.dtype, qs, st, lane);
    }
  }
  if (split == n_splits - 1) {
    const int len = cv.tail_len[layer * dm.batch + b];
    const long long tbase = ((static_cast<long long>(layer) * dm.batch + b) * dm.n_kv_heads + h) * dm.tail_capacity * kHeadDim;
    for (int t0 = warp * 32; t0 < len; t0 += kDecWarps * 32)
      process_raw_rows<G, false>(cv.tail_k + tbase + t0 * kHeadDim, cv.tail_v + tbase + t0 * kHeadDim,
                                 min(32, len - t0), dm.dtype, qs, st, lane);
  }

  // merge the warps of this CTA
#pragma unroll
  for (int g = 0; g < G; ++g) {
#pragma unroll
    for (int k = 0; k < 4; ++k) red_o[warp][g][4 * lane + k] = st.acc[g][k];
    if (lane == 0) { red_ml[warp][g][0] = st.m[g]; red_ml[warp][g][1] = st.l[g]; }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < G * kHeadDim; i += blockDim.x) {
    const int g = i / kHeadDim, c = i % kHeadDim;
    float m = -INFINITY;
#pragma unroll
    for (int wv = 0; wv < kDecWarps; ++wv) m = fmaxf(m, red_ml[wv][g][0]);
    float l = 0.0f, o = 0.0f;
#pragma unroll
    for (int wv = 0; wv < kDecWarps; ++wv) {
      const float f = (red_ml[wv][g][0] == -INFINITY) ? 0.0f : __expf(red_ml[wv][g][0] - m);
      l += red_ml[wv][g][1] * f;
      o += red_o[wv][g][c] * f;
    }
    const long long row = (static_cast<long long>(b) * dm.n_q_heads + h * G + g) * n_splits + split;
    ws_o[row * kHeadDim + c] = o;
    if (c == 0) { ws_ml[row * 2] = m; ws_ml[row * 2 + 1] = l; }
  }
}

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

template <int G>
cudaError_t launch_decode_g(const Dims& dm, const CacheView& cv, const void* q, int layer, float* out,
                            float scale, float* ws_o, float* ws_ml, int n_splits, cudaStream_t st) {
  dim3 grid(n_splits, dm.n_kv_heads, dm.batch);
  decode_splitk_kernel<G><<<grid, kDecWarps * 32, 0, st>>>(dm, cv, static_cast<const uint16_t*>(q), layer, scale,
                                                         ws_o, ws_ml, n_splits);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  decode_combine_kernel<<<dm.batch * dm.n_q_heads, kHeadDim, 0, st>>>(ws_o, ws_ml, out, n_splits);
  return cudaGetLastError();
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

cudaError_t launch_decode(const Dims& dm, const CacheView& cv, const void* q, int layer, float* out,
                          float scale, float* workspace, int n_splits, cudaStream_t st) {
  const long long rows = static_cast<long long>(dm.batch) * dm.n_q_heads * n_splits;
  float* ws_o = workspace;
  float* ws_ml = workspace + rows * kHeadDim;
  static const bool scalar = [] {
    const char* e = getenv("MOQAE_DECODE_KERNEL");      // "scalar": plain-FMA kernel, for debugging
    return e && e[0] == 's';
  }();
  if (!scalar) {
    cudaError_t e = launch_decode_mma(dm, cv, q, layer, scale, ws_o, ws_ml, n_splits, st);
    if (e != cudaSuccess) return e;
    decode_combine_kernel<<<dm.batch * dm.n_q_heads, kHeadDim, 0, st>>>(ws_o, ws_ml, out, n_splits);
    return cudaGetLastError();
  }
  switch (dm.n_q_heads / dm.n_kv_heads) {
    case 1: return launch_decode_g<1>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    case 2: return launch_decode_g<2>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    case 3: return launch_decode_g<3>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    case 4: return launch_decode_g<4>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    case 5: return launch_decode_g<5>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    case 6: return launch_decode_g<6>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    case 7: return launch_decode_g<7>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    case 8: return launch_decode_g<8>(dm, cv, q, layer, out, scale, ws_o, ws_ml, n_splits, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace moqae
