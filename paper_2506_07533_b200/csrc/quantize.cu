// Quantise + bit-pack kernels (prefill) and the 16-bit tail writers.
//
// quantize_pack_kernel: every warp is an independent tile pipeline.  A tile is 32 tokens x
// 128 channels of one kv head: 8 KiB of key rows and 8 KiB of value rows, each fetched by ONE
// tiled TMA copy (a 128 x 32 box of the [batch*T][heads*128] tensor) into the warp's own
// shared-memory buffers (mbarrier complete_tx), so the next tile's rows are in flight while
// the current one is encoded.
// The encoded tile (metadata + key payload + value payload, 3 / 5 / 9 KiB) is assembled in
// shared memory in its storage order and leaves with a single bulk store.  16-bit tiles are
// copied row by row with their 16-byte units swizzled.
//
// Arithmetic per element: binary32 subtract of the group's zero, then one fused
// multiply-add with 1/scale and the constant 1.5 * 2^23: the FMA rounds the exact product
// to the nearest integer (halves to even) and leaves the code in the low mantissa bits.
// HBM-bound by design: 512 B read and 96..512 B written per token and head.
#include "ptx.cuh"
#include "quant_encode.cuh"

namespace moqae {

namespace {

constexpr int kQWarps = 4;
constexpr int kInBytes = 8192;                 // 32 rows x 256 B
constexpr int kOutBytes = 9216;                // largest quantised tile
constexpr int kPrmBytes = 2048;                // value groups: [32 tokens][4 groups] (-zero, -zero, 1/scale, 1/scale)
constexpr int kWarpSmem = 2 * kInBytes + kOutBytes + kPrmBytes;
constexpr int kSkipTile = 0xfe;                // width marker: nothing to do for this tile

struct TileRef {
  int x, y;            // TMA coordinates: column h*128, token row b*T + c*chunk + j*32
  int b, j, h;
  int w, slot;         // routed width and slot of the tile's chunk
};

// FULL: every tile holds 32 tokens (chunk >= 32).  Chunks of 8 or 16 tokens get their own instantiation, so that
// the padding-row variants of the encoders do not take instruction-cache space in the ordinary kernel.
template <bool BF16, bool FULL>
__global__ void __launch_bounds__(kQWarps * 32, 2)
quantize_pack_kernel(Dims dm, CacheView cv, const __grid_constant__ CUtensorMap mapK,
                     const __grid_constant__ CUtensorMap mapV, int T, int layer, long long n_tiles, int flush) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint8_t* bufK = smem + warp * kWarpSmem;
  uint8_t* bufV = bufK + kInBytes;
  uint8_t* out = bufV + kInBytes;
  float4* prm = reinterpret_cast<float4*>(out + kOutBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kQWarps * kWarpSmem) + 2 * warp;
  const uint32_t barK = smem_u32(bars), barV = smem_u32(bars + 1);
  if (lane == 0) {
    mbar_init(barK, 1);
    mbar_init(barV, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncwarp();

  const int H = dm.n_kv_heads;
  const int tpc = tiles_per_chunk_of(dm.chunk);
  const int n_valid = tile_tokens_of(dm.chunk);      // rows of a tile that hold tokens (a short chunk: the rest is padding)
  constexpr bool full = FULL;
  const int C = T / dm.chunk;
  const long long stride = static_cast<long long>(gridDim.x) * kQWarps;
  const int group = layer / dm.rs_group;
  const uint8_t* map_g = cv.map + static_cast<long long>(group) * dm.n_tseq * dm.max_chunks;
  const int32_t* slot_g = cv.slot + static_cast<long long>(group) * dm.n_tseq * dm.max_chunks;

  const int32_t* count_g = cv.count + static_cast<long long>(group) * dm.batch * 4;
  // Tile id = ((b * Cd + c) * tpc + j) * H + h (heads fastest, so neighbouring warps read neighbouring
  // 256-byte segments of the same token rows); Cd = chunks per sequence (1 for a flush: one chunk per
  // sequence).  The id is taken apart by division once per warp; after that the four digits advance by
  // the digits of the grid stride with carries, which costs a dozen instructions per tile instead of
  // three 64-bit divisions.
  struct TilePos { int h, j, c, b; };
  const int Cd = flush ? 1 : C;
  auto split_id = [&](long long id) {
    TilePos p;
    p.h = static_cast<int>(id % H);
    long long x = id / H;
    p.j = static_cast<int>(x % tpc);
    x /= tpc;
    p.c = static_cast<int>(x % Cd);
    p.b = static_cast<int>(x / Cd);
    return p;
  };
  auto advance = [&](TilePos& p, const TilePos& d) {
    p.h += d.h;
    int carry = p.h >= H ? 1 : 0;
    p.h -= carry * H;
    p.j += d.j + carry;
    carry = p.j >= tpc ? 1 : 0;
    p.j -= carry * tpc;
    p.c += d.c + carry;
    carry = p.c >= Cd ? 1 : 0;
    p.c -= carry * Cd;
    p.b += d.b + carry;
  };
  auto tile_ref = [&](const TilePos& p) {
    TileRef r;
    r.h = p.h;
    r.j = p.j;
    if (!flush) {
      const int c = p.c;
      r.b = p.b;
      r.x = r.h * kHeadDim;
      r.y = r.b * T + c * dm.chunk + r.j * kTileTokens;
      const long long tbl = static_cast<long long>(table_row(dm, r.b, r.h)) * dm.max_chunks + c;
      r.w = map_g[tbl];                      // loaded one tile ahead of their use
      r.slot = slot_g[tbl];
    } else {
      // flush of a full tail: the source is the tail itself ([layer][b][h][row][128]); the target is
      // the sequence's newest chunk, marked with bit 7 in the map while its rows are being packed
      r.b = p.b;
      r.x = 0;
      r.y = ((layer * dm.batch + r.b) * H + r.h) * dm.tail_capacity + r.j * kTileTokens;
      const int c = count_g[4 * r.b] + count_g[4 * r.b + 1] + count_g[4 * r.b + 2] + count_g[4 * r.b + 3] - 1;
      r.w = kSkipTile;
      r.slot = 0;
      if (c >= 0) {
        const long long tbl = static_cast<long long>(r.b) * dm.max_chunks + c;
        const int e = map_g[tbl];
        if (e & 0x80) { r.w = e & 0x7f; r.slot = slot_g[tbl]; }
      }
    }
    return r;
  };
  auto fetch = [&](const CUtensorMap* map, const TileRef& r, uint8_t* buf, uint32_t bar) {
    if (lane == 0) {
      mbar_expect_tx(bar, kInBytes);
      tma_load_2d(smem_u32(buf), map, r.x, r.y, bar);
    }
  };

  long long id = static_cast<long long>(blockIdx.x) * kQWarps + warp;
  if (id >= n_tiles) return;
  TilePos pos = split_id(id);
  const TilePos step = split_id(stride);
  TileRef cur = tile_ref(pos);
  fetch(&mapK, cur, bufK, barK);
  fetch(&mapV, cur, bufV, barV);
  uint32_t parity = 0;
  bool store_pending = false;
  int failed = 0;                             // 1: key rows never arrived, 2: value rows

  for (; id < n_tiles; id += stride) {
    const long long next = id + stride;
    TileRef nxt = cur;
    if (next < n_tiles) {
      advance(pos, step);
      nxt = tile_ref(pos);
    }
    const int w = cur.w, slot = cur.slot;
    long long cap = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) cap = (w == k) ? cv.capacity[k] : cap;
    const bool valid = w <= 3 && slot >= 0 && slot < cap;
    if (!valid && w != kSkipTile && lane == 0) set_status(cv.status, MOQAE_ERR_POOL_FULL, w, slot);
    uint8_t* tile = nullptr;
    if (valid) {
      const long long tb = tile_bytes_of_expert(w);
      const long long idx = ((static_cast<long long>(layer) * dm.batch + cur.b) * H + cur.h) * cap + slot;
      uint8_t* pool = cv.pool[0];
#pragma unroll
      for (int k = 1; k < 4; ++k) pool = (w == k) ? cv.pool[k] : pool;
      tile = pool + (idx * tpc + cur.j) * tb;
    }

    // ---- keys
    if (!mbar_wait_bounded(barK, parity)) { failed = 1; break; }
    if (valid) {
      if (w == 3) {
        if constexpr (full) copy_raw_rows(bufK, tile, lane);
        else copy_raw_rows<true>(bufK, tile, lane, n_valid);
      } else {
        if (store_pending) {                  // the previous tile's bulk store must have read `out`
          if (lane == 0) bulk_store_wait_read();
          __syncwarp();
          store_pending = false;
        }
        if constexpr (full) {
          if (w == 0) encode_keys<2, BF16>(bufK, out, lane);
          else if (w == 1) encode_keys<4, BF16>(bufK, out, lane);
          else encode_keys<8, BF16>(bufK, out, lane);
        } else {                              // a chunk of 8 or 16 tokens: rows past it are padding
          if (w == 0) encode_keys<2, BF16, true>(bufK, out, lane, n_valid);
          else if (w == 1) encode_keys<4, BF16, true>(bufK, out, lane, n_valid);
          else encode_keys<8, BF16, true>(bufK, out, lane, n_valid);
        }
      }
    }
    __syncwarp();                             // every lane is done reading bufK
    if (next < n_tiles) fetch(&mapK, nxt, bufK, barK);

    // ---- values
    if (!mbar_wait_bounded(barV, parity)) { failed = 2; break; }
    if (valid) {
      if (w == 3) {
        if constexpr (full) copy_raw_rows(bufV, tile + 8192, lane);
        else copy_raw_rows<true>(bufV, tile + 8192, lane, n_valid);
      } else if constexpr (full) {
        if (w == 0) encode_values<2, BF16>(bufV, out, prm, lane);
        else if (w == 1) encode_values<4, BF16>(bufV, out, prm, lane);
        else encode_values<8, BF16>(bufV, out, prm, lane);
      } else {
        if (w == 0) encode_values<2, BF16, true>(bufV, out, prm, lane, n_valid);
        else if (w == 1) encode_values<4, BF16, true>(bufV, out, prm, lane, n_valid);
        else encode_values<8, BF16, true>(bufV, out, prm, lane, n_valid);
      }
    }
    __syncwarp();
    if (next < n_tiles) fetch(&mapV, nxt, bufV, barV);
    if (valid && w != 3) {
      fence_async_smem();                     // generic-proxy writes to `out` -> visible to the bulk store
      __syncwarp();
      if (lane == 0) bulk_store(tile, smem_u32(out), tile_bytes_of_expert(w));
      store_pending = true;
    }
    parity ^= 1u;
    cur = nxt;
  }
  if (failed) {
    // a copy did not land in time: report it, then give the copies still in flight a last
    // bounded chance to finish before this CTA's shared memory goes away
    if (lane == 0) set_status(cv.status, MOQAE_ERR_TIMEOUT, blockIdx.x, warp);
    if (failed == 1) {
      mbar_wait_bounded(barK, parity);
      mbar_wait_bounded(barV, parity);
    } else {
      if (id + stride < n_tiles) mbar_wait_bounded(barK, parity ^ 1u);   // next tile's key rows
      mbar_wait_bounded(barV, parity);
    }
  }
  if (lane == 0) bulk_store_wait_all();
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

__global__ void flush_reset_kernel(Dims dm, CacheView cv, int group) {
  const int b = blockIdx.x;
  const int32_t* count = cv.count + (static_cast<long long>(group) * dm.batch + b) * 4;
  const int c = count[0] + count[1] + count[2] + count[3] - 1;
  if (c < 0) return;
  uint8_t* entry = cv.map + (static_cast<long long>(group) * dm.batch + b) * dm.max_chunks + c;
  if (!(*entry & 0x80)) return;
  __syncwarp();
  if (threadIdx.x == 0) *entry &= 0x7f;
  for (int l = group * dm.rs_group + threadIdx.x; l < min(dm.n_layers, (group + 1) * dm.rs_group); l += 32)
    cv.tail_len[l * dm.batch + b] = 0;
}

int sm_count() { return sm_count_of_current_device(); }

}  // namespace
// [rows][cols] 16-bit tensor, boxes of 128 columns x 32 rows (one tile), no swizzle
static bool make_tile_map(CUtensorMap* m, const void* base, long long rows, long long cols) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(cols) * 2};
  const cuuint32_t box[2] = {kHeadDim, kTileTokens};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool BF16, bool FULL>
static cudaError_t launch_quantize_pack_t(const Dims& dm, const CacheView& cv, const CUtensorMap& mapK, const CUtensorMap& mapV,
                                          int T, int layer, long long n_tiles, int flush, unsigned grid, size_t smem,
                                          cudaStream_t st) {
  const cudaError_t e = cudaFuncSetAttribute(quantize_pack_kernel<BF16, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  quantize_pack_kernel<BF16, FULL><<<grid, kQWarps * 32, smem, st>>>(dm, cv, mapK, mapV, T, layer, n_tiles, flush);
  return cudaGetLastError();
}

// one instantiation per (input dtype, whole tiles / chunks shorter than a tile)
static cudaError_t launch_quantize_pack(const Dims& dm, const CacheView& cv, const CUtensorMap& mapK, const CUtensorMap& mapV,
                                        int T, int layer, long long n_tiles, int flush, unsigned grid, size_t smem,
                                        cudaStream_t st) {
  const bool bf16 = dm.dtype == MOQAE_DTYPE_BF16, full = tile_tokens_of(dm.chunk) == kTileTokens;
  if (bf16) return full ? launch_quantize_pack_t<true, true>(dm, cv, mapK, mapV, T, layer, n_tiles, flush, grid, smem, st)
                        : launch_quantize_pack_t<true, false>(dm, cv, mapK, mapV, T, layer, n_tiles, flush, grid, smem, st);
  return full ? launch_quantize_pack_t<false, true>(dm, cv, mapK, mapV, T, layer, n_tiles, flush, grid, smem, st)
              : launch_quantize_pack_t<false, false>(dm, cv, mapK, mapV, T, layer, n_tiles, flush, grid, smem, st);
}

cudaError_t launch_quantize(const Dims& dm, const CacheView& cv, const void* K, const void* V, int T,
                            int layer, cudaStream_t st) {
  const int C = T / dm.chunk;
  const long long n_tiles = static_cast<long long>(dm.batch) * C * tiles_per_chunk_of(dm.chunk) * dm.n_kv_heads;
  if (n_tiles > 0) {
    CUtensorMap mapK, mapV;
    const long long rows = static_cast<long long>(dm.batch) * T, cols = static_cast<long long>(dm.n_kv_heads) * kHeadDim;
    if (!make_tile_map(&mapK, K, rows, cols) || !make_tile_map(&mapV, V, rows, cols)) return cudaErrorNotSupported;
    const size_t smem = static_cast<size_t>(kQWarps) * kWarpSmem + kQWarps * 16;
    const long long want = (n_tiles + kQWarps - 1) / kQWarps;
    const long long cap = 2ll * sm_count();                    // two resident CTAs per SM, grid-stride
    const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
    const cudaError_t e = launch_quantize_pack(dm, cv, mapK, mapV, T, layer, n_tiles, 0, grid, smem, st);
    if (e != cudaSuccess) return e;
  }
  dim3 g(8, dm.batch);
  tail_copy_kernel<<<g, 256, 0, st>>>(dm, cv, static_cast<const uint16_t*>(K), static_cast<const uint16_t*>(V), T, layer);
  return cudaGetLastError();
}

// Pack the full tails of `layer` into the chunk that launch_flush_route has just added to the tables.
cudaError_t launch_flush_quantize(const Dims& dm, const CacheView& cv, int layer, cudaStream_t st) {
  const long long n_tiles = static_cast<long long>(dm.batch) * tiles_per_chunk_of(dm.chunk) * dm.n_kv_heads;
  CUtensorMap mapK, mapV;
  const long long rows = static_cast<long long>(dm.n_layers) * dm.batch * dm.n_kv_heads * dm.tail_capacity;
  if (!make_tile_map(&mapK, cv.tail_k, rows, kHeadDim) || !make_tile_map(&mapV, cv.tail_v, rows, kHeadDim))
    return cudaErrorNotSupported;
  const size_t smem = static_cast<size_t>(kQWarps) * kWarpSmem + kQWarps * 16;
  const long long want = (n_tiles + kQWarps - 1) / kQWarps;
  const long long cap = 2ll * sm_count();
  const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
  return launch_quantize_pack(dm, cv, mapK, mapV, 0, layer, n_tiles, 1, grid, smem, st);
}

// After every layer of the group has packed its rows: clear the marker and empty the tails.
cudaError_t launch_flush_reset(const Dims& dm, const CacheView& cv, int group, cudaStream_t st) {
  flush_reset_kernel<<<dm.batch, 32, 0, st>>>(dm, cv, group);
  return cudaGetLastError();
}

cudaError_t launch_append(const Dims& dm, const CacheView& cv, const void* k_new, const void* v_new,
                          int layer, cudaStream_t st) {
  append_kernel<<<dm.batch, 128, 0, st>>>(dm, cv, static_cast<const uint16_t*>(k_new),
                                          static_cast<const uint16_t*>(v_new), layer);
  return cudaGetLastError();
}

}  // namespace moqae
