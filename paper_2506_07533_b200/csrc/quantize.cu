// Quantise + bit-pack kernels: one warp owns one tile (32 tokens x 128 channels of one kv
// head), computes the group statistics, the integer codes and the packed words, and stores
// them into the slot of the tile's chunk.  HBM-bound: 512 B read and 96..512 B written per
// token and head.
#include "common.cuh"

namespace moqae {

namespace {

constexpr int kWarpsPerBlock = 4;

__device__ __forceinline__ float cvt16(uint32_t u, int dtype) {
  return load16_as_float(static_cast<uint16_t>(u), dtype);
}

// Group parameters from min / max, every step one binary32 operation.
__device__ __forceinline__ void group_params(float mn, float mx, float qmax, __half& s, __half& z,
                                             float& zf, float& inv, bool& dead) {
  z = __float2half_rd(mn);
  zf = __half2float(z);
  const float r = __fsub_rn(mx, zf);
  s = __float2half_ru(__fdiv_rn(r, qmax));
  const float sf = __half2float(s);
  dead = (sf == 0.0f);
  inv = __frcp_rn(sf);
}

__device__ __forceinline__ uint32_t encode(float x, float zf, float inv, float qmax, bool dead) {
  float c = rintf(__fmul_rn(__fsub_rn(x, zf), inv));
  c = fminf(qmax, fmaxf(0.0f, c));
  return dead ? 0u : static_cast<uint32_t>(c);
}

// Partial 32-bit word of the four positions 4*vl .. 4*vl+3 of a row.
template <int BITS>
__device__ __forceinline__ uint32_t place4(const uint32_t c[4], int vl) {
  constexpr int n = 32 / BITS;
  const int i0 = (4 * vl) & (n - 1);
  uint32_t w = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int i = i0 + j;
    w |= c[j] << (BITS * (i >> 1) + 16 * (i & 1));
  }
  return w;
}

// Store one row word: `vl` is the virtual lane (positions 4*vl..4*vl+3), `xor_a/xor_b` the
// physical-lane distances of the lanes that share a word.
template <int BITS>
__device__ __forceinline__ void store_row_word(uint8_t* payload, int t, int vl, uint32_t part, int xor_a,
                                               int xor_b) {
  constexpr int lanes_per_word = (32 / BITS) / 4;   // 4, 2, 1
  if (lanes_per_word >= 2) part |= __shfl_xor_sync(0xffffffffu, part, xor_a);
  if (lanes_per_word >= 4) part |= __shfl_xor_sync(0xffffffffu, part, xor_b);
  const int wj = vl / lanes_per_word;
  int unit = wj >> 2;
  if (BITS == 8) unit ^= (t & 7);
  if ((vl % lanes_per_word) == 0)
    *reinterpret_cast<uint32_t*>(payload + t * 16 * BITS + unit * 16 + (wj & 3) * 4) = part;
}

template <int BITS>
__device__ void quantize_tile(const uint16_t* __restrict__ Kg, const uint16_t* __restrict__ Vg,
                              long long row_stride, uint8_t* __restrict__ tile, int dtype, int lane) {
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  uint2 raw[kTileTokens];

  // ---- keys: one group per channel over the 32 tokens; this lane owns channels 4*lane..+3
#pragma unroll
  for (int t = 0; t < kTileTokens; ++t)
    raw[t] = __ldg(reinterpret_cast<const uint2*>(Kg + t * row_stride) + lane);
  float mn[4], mx[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) { mn[j] = INFINITY; mx[j] = -INFINITY; }
#pragma unroll
  for (int t = 0; t < kTileTokens; ++t) {
    const float x0 = cvt16(raw[t].x & 0xffffu, dtype), x1 = cvt16(raw[t].x >> 16, dtype);
    const float x2 = cvt16(raw[t].y & 0xffffu, dtype), x3 = cvt16(raw[t].y >> 16, dtype);
    mn[0] = fminf(mn[0], x0); mx[0] = fmaxf(mx[0], x0);
    mn[1] = fminf(mn[1], x1); mx[1] = fmaxf(mx[1], x1);
    mn[2] = fminf(mn[2], x2); mx[2] = fmaxf(mx[2], x2);
    mn[3] = fminf(mn[3], x3); mx[3] = fmaxf(mx[3], x3);
  }
  {
    float zf[4], inv[4];
    bool dead[4];
    __half s[4], z[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) group_params(mn[j], mx[j], qmax, s[j], z[j], zf[j], inv[j], dead[j]);
    uint2 ps, pz;
    ps.x = __half_as_ushort(s[0]) | (static_cast<uint32_t>(__half_as_ushort(s[1])) << 16);
    ps.y = __half_as_ushort(s[2]) | (static_cast<uint32_t>(__half_as_ushort(s[3])) << 16);
    pz.x = __half_as_ushort(z[0]) | (static_cast<uint32_t>(__half_as_ushort(z[1])) << 16);
    pz.y = __half_as_ushort(z[2]) | (static_cast<uint32_t>(__half_as_ushort(z[3])) << 16);
    reinterpret_cast<uint2*>(tile)[lane] = ps;
    reinterpret_cast<uint2*>(tile + 256)[lane] = pz;
    uint8_t* payload = tile + kMetaBytes;
#pragma unroll
    for (int t = 0; t < kTileTokens; ++t) {
      uint32_t c[4];
      c[0] = encode(cvt16(raw[t].x & 0xffffu, dtype), zf[0], inv[0], qmax, dead[0]);
      c[1] = encode(cvt16(raw[t].x >> 16, dtype), zf[1], inv[1], qmax, dead[1]);
      c[2] = encode(cvt16(raw[t].y & 0xffffu, dtype), zf[2], inv[2], qmax, dead[2]);
      c[3] = encode(cvt16(raw[t].y >> 16, dtype), zf[3], inv[3], qmax, dead[3]);
      store_row_word<BITS>(payload, t, lane, place4<BITS>(c, lane), 1, 2);
    }
  }

  // ---- values: one group per token over 32 channels = 8 lanes (lane>>3 is the channel group)
#pragma unroll
  for (int t = 0; t < kTileTokens; ++t)
    raw[t] = __ldg(reinterpret_cast<const uint2*>(Vg + t * row_stride) + lane);
  const int cg = lane >> 3, u = lane & 7;
  const int vl = 4 * u + cg;                       // value rows are stored channel-group interleaved
  uint8_t* payload = tile + kMetaBytes + kTileTokens * 16 * BITS;
  __half keep_s[4], keep_z[4];
#pragma unroll
  for (int t = 0; t < kTileTokens; ++t) {
    const float x0 = cvt16(raw[t].x & 0xffffu, dtype), x1 = cvt16(raw[t].x >> 16, dtype);
    const float x2 = cvt16(raw[t].y & 0xffffu, dtype), x3 = cvt16(raw[t].y >> 16, dtype);
    float lo = fminf(fminf(x0, x1), fminf(x2, x3));
    float hi = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
#pragma unroll
    for (int m = 1; m <= 4; m <<= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, m));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, m));
    }
    __half s, z;
    float zf, inv;
    bool dead;
    group_params(lo, hi, qmax, s, z, zf, inv, dead);
    if ((t & 7) == u) { keep_s[t >> 3] = s; keep_z[t >> 3] = z; }
    uint32_t c[4];
    c[0] = encode(x0, zf, inv, qmax, dead);
    c[1] = encode(x1, zf, inv, qmax, dead);
    c[2] = encode(x2, zf, inv, qmax, dead);
    c[3] = encode(x3, zf, inv, qmax, dead);
    store_row_word<BITS>(payload, t, vl, place4<BITS>(c, vl), 8, 16);
  }
  __half* vs = reinterpret_cast<__half*>(tile + 512) + cg * 32;
  __half* vz = reinterpret_cast<__half*>(tile + 768) + cg * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    vs[8 * i + u] = keep_s[i];
    vz[8 * i + u] = keep_z[i];
  }
}

// 16-bit tile: rows are copied in the input dtype with 16-byte units swizzled.
__device__ void copy_raw_tile(const uint16_t* __restrict__ Kg, const uint16_t* __restrict__ Vg,
                              long long row_stride, uint8_t* __restrict__ tile, int lane) {
  const int U = lane >> 1;
#pragma unroll 8
  for (int t = 0; t < kTileTokens; ++t) {
    const uint2 k = __ldg(reinterpret_cast<const uint2*>(Kg + t * row_stride) + lane);
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(Vg + t * row_stride) + lane);
    const int up = (U & 8) | ((U ^ t) & 7);
    const int off = t * 256 + up * 16 + (lane & 1) * 8;
    *reinterpret_cast<uint2*>(tile + off) = k;
    *reinterpret_cast<uint2*>(tile + 8192 + off) = v;
  }
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
quantize_pack_kernel(Dims dm, CacheView cv, const uint16_t* __restrict__ K, const uint16_t* __restrict__ V,
                     int T, int layer, long long n_tiles) {
  const int lane = threadIdx.x & 31;
  const long long tile_id = static_cast<long long>(blockIdx.x) * kWarpsPerBlock + (threadIdx.x >> 5);
  if (tile_id >= n_tiles) return;
  const int H = dm.n_kv_heads;
  const int tpc = dm.chunk / kTileTokens;
  const int C = T / dm.chunk;
  // tile_id = ((b * C + c) * tpc + j) * H + h : heads fastest, so neighbouring warps read
  // neighbouring 256-byte segments of the same token rows
  const int h = static_cast<int>(tile_id % H);
  long long r = tile_id / H;
  const int j = static_cast<int>(r % tpc);
  r /= tpc;
  const int c = static_cast<int>(r % C);
  const int b = static_cast<int>(r / C);
  const int group = layer / dm.rs_group;
  const long long tbl = (static_cast<long long>(group) * dm.batch + b) * dm.max_chunks + c;
  const int w = cv.map[tbl];
  const int slot = cv.slot[tbl];
  if (w > 3 || slot < 0 || slot >= cv.capacity[w > 3 ? 0 : w]) {
    if (lane == 0) set_status(cv.status, MOQAE_ERR_POOL_FULL, w, slot);
    return;
  }
  const long long row_stride = static_cast<long long>(H) * kHeadDim;
  const long long tok0 = static_cast<long long>(b) * T + static_cast<long long>(c) * dm.chunk + j * kTileTokens;
  const uint16_t* Kg = K + tok0 * row_stride + h * kHeadDim;
  const uint16_t* Vg = V + tok0 * row_stride + h * kHeadDim;
  uint8_t* tile = slot_ptr(cv, dm, w, layer, b, h, slot) + static_cast<long long>(j) * tile_bytes_of_expert(w);
  switch (w) {
    case 0: quantize_tile<2>(Kg, Vg, row_stride, tile, dm.dtype, lane); break;
    case 1: quantize_tile<4>(Kg, Vg, row_stride, tile, dm.dtype, lane); break;
    case 2: quantize_tile<8>(Kg, Vg, row_stride, tile, dm.dtype, lane); break;
    default: copy_raw_tile(Kg, Vg, row_stride, tile, lane); break;
  }
}

// Trailing T mod chunk tokens -> tail rows [layer][b][h][t][128]; sets tail_len.
__global__ void tail_copy_kernel(Dims dm, CacheView cv, const uint16_t* __restrict__ K,
                                 const uint16_t* __restrict__ V, int T, int layer) {
  const int b = blockIdx.y;
  const int C = T / dm.chunk;
  const int r = T - C * dm.chunk;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (r > dm.tail_capacity) set_status(cv.status, MOQAE_ERR_POOL_FULL, -1, r);
    cv.tail_len[layer * dm.batch + b] = min(r, dm.tail_capacity);
  }
  const int rows = min(r, dm.tail_capacity);
  const int H = dm.n_kv_heads;
  const long long total = static_cast<long long>(rows) * H * (kHeadDim / 8);   // 16-byte pieces
  for (long long i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int piece = static_cast<int>(i % (kHeadDim / 8));
    long long q = i / (kHeadDim / 8);
    const int h = static_cast<int>(q % H);
    const int t = static_cast<int>(q / H);
    const long long src = ((static_cast<long long>(b) * T + C * static_cast<long long>(dm.chunk) + t) * H + h) * kHeadDim + piece * 8;
    const long long dst = (((static_cast<long long>(layer) * dm.batch + b) * H + h) * dm.tail_capacity + t) * kHeadDim + piece * 8;
    *reinterpret_cast<uint4*>(cv.tail_k + dst) = __ldg(reinterpret_cast<const uint4*>(K + src));
    *reinterpret_cast<uint4*>(cv.tail_v + dst) = __ldg(reinterpret_cast<const uint4*>(V + src));
  }
}

__global__ void append_kernel(Dims dm, CacheView cv, const uint16_t* __restrict__ k_new,
                              const uint16_t* __restrict__ v_new, int layer) {
  const int b = blockIdx.x;
  const int len = cv.tail_len[layer * dm.batch + b];
  if (len >= dm.tail_capacity) {
    if (threadIdx.x == 0) set_status(cv.status, MOQAE_ERR_POOL_FULL, -2, len);
    return;
  }
  const int H = dm.n_kv_heads;
  for (int i = threadIdx.x; i < H * (kHeadDim / 8); i += blockDim.x) {
    const int h = i / (kHeadDim / 8), piece = i % (kHeadDim / 8);
    const long long src = (static_cast<long long>(b) * H + h) * kHeadDim + piece * 8;
    const long long dst = (((static_cast<long long>(layer) * dm.batch + b) * H + h) * dm.tail_capacity + len) * kHeadDim + piece * 8;
    *reinterpret_cast<uint4*>(cv.tail_k + dst) = __ldg(reinterpret_cast<const uint4*>(k_new + src));
    *reinterpret_cast<uint4*>(cv.tail_v + dst) = __ldg(reinterpret_cast<const uint4*>(v_new + src));
  }
  __syncthreads();
  if (threadIdx.x == 0) cv.tail_len[layer * dm.batch + b] = len + 1;
}

}  // namespace

cudaError_t launch_quantize(const Dims& dm, const CacheView& cv, const void* K, const void* V, int T,
                            int layer, cudaStream_t st) {
  const int C = T / dm.chunk;
  const long long n_tiles = static_cast<long long>(dm.batch) * C * (dm.chunk / kTileTokens) * dm.n_kv_heads;
  if (n_tiles > 0) {
    const long long blocks = (n_tiles + kWarpsPerBlock - 1) / kWarpsPerBlock;
    quantize_pack_kernel<<<static_cast<unsigned>(blocks), kWarpsPerBlock * 32, 0, st>>>(
        dm, cv, static_cast<const uint16_t*>(K), static_cast<const uint16_t*>(V), T, layer, n_tiles);
  }
  dim3 g(8, dm.batch);
  tail_copy_kernel<<<g, 256, 0, st>>>(dm, cv, static_cast<const uint16_t*>(K), static_cast<const uint16_t*>(V), T, layer);
  return cudaGetLastError();
}

cudaError_t launch_append(const Dims& dm, const CacheView& cv, const void* k_new, const void* v_new,
                          int layer, cudaStream_t st) {
  append_kernel<<<dm.batch, 128, 0, st>>>(dm, cv, static_cast<const uint16_t*>(k_new),
                                          static_cast<const uint16_t*>(v_new), layer);
  return cudaGetLastError();
}

}  // namespace moqae
