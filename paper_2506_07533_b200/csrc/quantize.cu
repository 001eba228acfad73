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
#include <cuda.h>

#include "common.cuh"

namespace moqae {

namespace {

constexpr int kQWarps = 4;
constexpr int kInBytes = 8192;                 // 32 rows x 256 B
constexpr int kOutBytes = 9216;                // largest quantised tile
constexpr int kPrmBytes = 2048;                // value groups: [32 tokens][4 groups] (-zero, -zero, 1/scale, 1/scale)
constexpr int kWarpSmem = 2 * kInBytes + kOutBytes + kPrmBytes;
constexpr long long kWaitCycles = 1ll << 30;  // a bounded wait gives up after this many SM cycles
constexpr uint32_t kSuspendNs = 20000;         // how long one try_wait may keep the warp parked
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23
constexpr int kSkipTile = 0xfe;                // width marker: nothing to do for this tile

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
// tiled TMA load of the box whose corner is (x = element column, y = token row)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
               ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory");
}
__device__ __forceinline__ void fence_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
}
// One try_wait with a suspend-time hint: the hardware parks the warp until the phase completes
// or the hint runs out, so a waiting warp takes no issue slots from the working ones.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendNs) : "memory");
  return ok != 0;
}
// Bounded by elapsed SM cycles (about half a second), not by the number of attempts.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  do {
    if (mbar_try_wait(bar, parity)) return true;
  } while (clock64() - t0 < kWaitCycles);
  return false;
}

// ---- packed 16-bit min / max (exact: comparisons only) ---------------------------------
template <bool BF16> __device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) {
  uint32_t d;
  if (BF16) asm("min.bf16x2 %0, %1, %2;\n" : "=r"(d) : "r"(a), "r"(b));
  else asm("min.f16x2 %0, %1, %2;\n" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
template <bool BF16> __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
  uint32_t d;
  if (BF16) asm("max.bf16x2 %0, %1, %2;\n" : "=r"(d) : "r"(a), "r"(b));
  else asm("max.f16x2 %0, %1, %2;\n" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
template <bool BF16> __device__ __forceinline__ float lo_f(uint32_t w) {
  if (BF16) return __uint_as_float(w << 16);
  return __low2float(*reinterpret_cast<const __half2*>(&w));
}
template <bool BF16> __device__ __forceinline__ float hi_f(uint32_t w) {
  if (BF16) return __uint_as_float(w & 0xffff0000u);
  return __high2float(*reinterpret_cast<const __half2*>(&w));
}

// Group parameters from min / max.  zf = stored zero as float, inv = 1/scale (0 for a
// constant group, so that every code comes out 0).
__device__ __forceinline__ void group_params(float mn, float mx, float qmax, uint16_t& s_bits, uint16_t& z_bits,
                                             float& zf, float& inv) {
  uint16_t zb = __half_as_ushort(__float2half_rd(mn));
  if (zb == 0x8000u) zb = 0;                                   // -0 is stored as +0
  zf = __half2float(__ushort_as_half(zb));
  const float r = __fsub_rn(mx, zf);
  const __half s = __float2half_ru(__fdiv_rn(r, qmax));
  const float sf = __half2float(s);
  inv = (sf == 0.0f) ? 0.0f : __frcp_rn(sf);
  s_bits = __half_as_ushort(s);
  z_bits = zb;
}

// code + 0x4B400000 = fma(x - z, inv, 1.5 * 2^23): the low bits of the result hold
// rint((x - z) * inv).  Done for the two 16-bit values of one word at once, as packed fp32 pairs
// (add.rn.f32x2 and fma.rn.f32x2 round each lane exactly like the scalar instructions; x + (-z)
// is x - z).
// negz2 = (-z_lo, -z_hi), inv2 = (inv_lo, inv_hi) as 64-bit register pairs.
__device__ __forceinline__ uint64_t pack_f2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
template <bool BF16>
__device__ __forceinline__ void encode2(uint32_t w, uint64_t negz2, uint64_t inv2, uint32_t& u_lo, uint32_t& u_hi) {
  const uint64_t x2 = pack_f2(lo_f<BF16>(w), hi_f<BF16>(w));
  uint64_t d2, r2;
  asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d2) : "l"(x2), "l"(negz2));
  asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(r2) : "l"(d2), "l"(inv2), "l"(pack_f2(kMagic, kMagic)));
  asm("mov.b64 {%0, %1}, %2;\n" : "=r"(u_lo), "=r"(u_hi) : "l"(r2));
}

// Four codes of `BITS` bits side by side in the low 4*BITS bits (higher bits: don't care for
// BITS < 8, exact for BITS == 8).
template <int BITS>
__device__ __forceinline__ uint32_t pack4(uint32_t u0, uint32_t u1, uint32_t u2, uint32_t u3) {
  if (BITS == 8) return __byte_perm(__byte_perm(u0, u1, 0x0040), __byte_perm(u2, u3, 0x0040), 0x5410);
  return u0 + (u1 << BITS) + (u2 << (2 * BITS)) + (u3 << (3 * BITS));
}

// halfword index of channel c in the key scale / zero arrays (register order of the decoder)
template <int BITS> __device__ __forceinline__ int key_meta_index(int c) {
  constexpr int n = 32 / BITS;
  const int q = c >> 5, cc = c & 31;
  const int j = cc / n, i = cc % n;
  const int hi = i >= n / 2 ? 1 : 0, i2 = i % (n / 2);
  const int s = i2 / (n / 4), m = i2 % (n / 4);
  const int r = j * (n / 2) + s * (n / 4) + m;
  return ((r >> 2) * 4 + q) * 8 + (r & 3) * 2 + hi;
}

// ---- keys: lane owns channels 4*lane .. 4*lane+3 over the tile's 32 tokens --------------
template <int BITS, bool BF16>
__device__ __forceinline__ void encode_keys(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, int lane) {
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  const uint2* rows = reinterpret_cast<const uint2*>(in) + lane;         // row t at rows[32 * t]
  uint32_t mn01, mn23, mx01, mx23;
  {
    const uint2 w = rows[0];
    mn01 = mx01 = w.x; mn23 = mx23 = w.y;
  }
#pragma unroll
  for (int t = 1; t < kTileTokens; ++t) {
    const uint2 w = rows[32 * t];
    mn01 = min2<BF16>(mn01, w.x); mx01 = max2<BF16>(mx01, w.x);
    mn23 = min2<BF16>(mn23, w.y); mx23 = max2<BF16>(mx23, w.y);
  }
  float zf[4], inv[4];
  uint16_t sb[4], zb[4];
  group_params(lo_f<BF16>(mn01), lo_f<BF16>(mx01), qmax, sb[0], zb[0], zf[0], inv[0]);
  group_params(hi_f<BF16>(mn01), hi_f<BF16>(mx01), qmax, sb[1], zb[1], zf[1], inv[1]);
  group_params(lo_f<BF16>(mn23), lo_f<BF16>(mx23), qmax, sb[2], zb[2], zf[2], inv[2]);
  group_params(hi_f<BF16>(mn23), hi_f<BF16>(mx23), qmax, sb[3], zb[3], zf[3], inv[3]);
  uint16_t* meta = reinterpret_cast<uint16_t*>(out);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int idx = key_meta_index<BITS>(4 * lane + k);
    meta[idx] = sb[k];
    // zeros: inside each group of four registers the order is 0, 2, 1, 3 (bits 1 and 2 of the index swap)
    meta[128 + ((idx & ~6) | ((idx & 2) << 1) | ((idx & 4) >> 1))] = zb[k];
  }
  // payload: this lane's 4 codes of token t are 4*BITS contiguous bits of the (t, quarter) piece
  uint8_t* pay = out + kMetaBytes;
  const uint64_t negz01 = pack_f2(-zf[0], -zf[1]), negz23 = pack_f2(-zf[2], -zf[3]);
  const uint64_t inv01 = pack_f2(inv[0], inv[1]), inv23 = pack_f2(inv[2], inv[3]);
  const int q = lane >> 3, l7 = lane & 7;
#pragma unroll
  for (int t = 0; t < kTileTokens; ++t) {
    const uint2 w = rows[32 * t];
    uint32_t u0, u1, u2, u3;
    encode2<BF16>(w.x, negz01, inv01, u0, u1);
    encode2<BF16>(w.y, negz23, inv23, u2, u3);
    const uint32_t p = pack4<BITS>(u0, u1, u2, u3);
    const int blk = t >> 4, hh = (t >> 3) & 1, g = t & 7;
    if (BITS == 2) {
      pay[(32 * blk + 4 * g + q) * 16 + 8 * hh + l7] = static_cast<uint8_t>(p);
    } else if (BITS == 4) {
      *reinterpret_cast<uint16_t*>(pay + (32 * (2 * blk + hh) + 4 * g + q) * 16 + 2 * l7) = static_cast<uint16_t>(p);
    } else {
      *reinterpret_cast<uint32_t*>(pay + (32 * (2 * (2 * blk + hh) + (l7 >> 2)) + 4 * g + q) * 16 + 4 * (l7 & 3)) = p;
    }
  }
}

// ---- values: groups are 32 channels of one token -----------------------------------------
template <int BITS, bool BF16>
__device__ __forceinline__ void encode_values(const uint8_t* __restrict__ in, uint8_t* __restrict__ out,
                                              float4* __restrict__ prm, int lane) {
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  uint16_t* meta = reinterpret_cast<uint16_t*>(out);
  {
    // statistics: lane = token; its row is read in 16-byte units, rotated inside each channel
    // group so that neighbouring lanes start on different banks
    const int t = lane;
    const uint4* row = reinterpret_cast<const uint4*>(in + t * 256);
    const int blk = t >> 4, half = (t >> 3) & 1, t4 = (t >> 1) & 3, e = t & 1;
#pragma unroll
    for (int cg = 0; cg < 4; ++cg) {
      uint32_t mn = 0, mx = 0;
#pragma unroll
      for (int ii = 0; ii < 4; ++ii) {
        const uint4 v = row[4 * cg + (ii ^ (t & 3))];
        const uint32_t a = min2<BF16>(min2<BF16>(v.x, v.y), min2<BF16>(v.z, v.w));
        const uint32_t b = max2<BF16>(max2<BF16>(v.x, v.y), max2<BF16>(v.z, v.w));
        mn = ii == 0 ? a : min2<BF16>(mn, a);
        mx = ii == 0 ? b : max2<BF16>(mx, b);
      }
      float zf, inv;
      uint16_t sb, zb;
      group_params(fminf(lo_f<BF16>(mn), hi_f<BF16>(mn)), fmaxf(lo_f<BF16>(mx), hi_f<BF16>(mx)), qmax, sb, zb, zf, inv);
      prm[4 * t + cg] = make_float4(-zf, -zf, inv, inv);
      meta[256 + ((((blk * 2 + (cg >> 1)) * 4 + t4) * 4 + (cg & 1) * 2 + half) * 2) + e] = sb;
      meta[384 + ((((blk * 4 + cg) * 4 + t4) * 2 + half) * 2) + e] = zb;
    }
  }
  __syncwarp();
  // codes: lane = channels 4*lane .. 4*lane+3 (group p = lane / 8); one word set per 4 tokens
  const int p = lane >> 3, g = lane & 7;
  const uint2* rows = reinterpret_cast<const uint2*>(in) + lane;
  uint8_t* pay = out + kMetaBytes + kTileTokens * 16 * BITS;
#pragma unroll
  for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
    for (int t4 = 0; t4 < 4; ++t4) {
      uint32_t u[4][4];                      // [byte position half + 2e][channel]
#pragma unroll
      for (int bp = 0; bp < 4; ++bp) {
        const int t = 16 * blk + 8 * (bp & 1) + 2 * t4 + (bp >> 1);
        const uint2 w = rows[32 * t];
        const ulonglong2 zi = *reinterpret_cast<const ulonglong2*>(prm + 4 * t + p);    // (-z, -z), (inv, inv)
        encode2<BF16>(w.x, zi.x, zi.y, u[bp][0], u[bp][1]);
        encode2<BF16>(w.y, zi.x, zi.y, u[bp][2], u[bp][3]);
      }
      const int ln = 4 * g + t4;
      if (BITS == 2) {
        uint32_t b[4];
#pragma unroll
        for (int bp = 0; bp < 4; ++bp) b[bp] = pack4<2>(u[bp][0], u[bp][1], u[bp][2], u[bp][3]);
        const uint32_t word = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
        *reinterpret_cast<uint32_t*>(pay + (blk * 32 + ln) * 16 + p * 4) = word;
      } else if (BITS == 4) {
        uint32_t word[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          uint32_t b[4];
#pragma unroll
          for (int bp = 0; bp < 4; ++bp) b[bp] = u[bp][2 * k] + (u[bp][2 * k + 1] << 4);
          word[k] = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
        }
        // words w = 2p, 2p+1 of the lane: unit w/4 = p/2, position 2*(p&1)
        *reinterpret_cast<uint2*>(pay + ((blk * 2 + (p >> 1)) * 32 + ln) * 16 + (p & 1) * 8) = make_uint2(word[0], word[1]);
      } else {
        uint4 word;
        uint32_t* wp = reinterpret_cast<uint32_t*>(&word);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          wp[k] = __byte_perm(__byte_perm(u[0][k], u[1][k], 0x0040), __byte_perm(u[2][k], u[3][k], 0x0040), 0x5410);
        *reinterpret_cast<uint4*>(pay + ((blk * 4 + p) * 32 + ln) * 16) = word;      // words 4p .. 4p+3
      }
    }
  }
}

// 16-bit tile half (keys or values): rows copied in the input dtype, 16-byte units swizzled.
__device__ __forceinline__ void copy_raw_rows(const uint8_t* __restrict__ in, uint8_t* __restrict__ dst, int lane) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int idx = i * 32 + lane;
    const int row = idx >> 4, U = idx & 15;
    const int up = (U & 8) | ((U ^ row) & 7);
    *reinterpret_cast<uint4*>(dst + row * 256 + up * 16) = *reinterpret_cast<const uint4*>(in + row * 256 + U * 16);
  }
}

struct TileRef {
  int x, y;            // TMA coordinates: column h*128, token row b*T + c*chunk + j*32
  int b, j, h;
  int w, slot;         // routed width and slot of the tile's chunk
};

template <bool BF16>
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
  const int tpc = dm.chunk / kTileTokens;
  const int C = T / dm.chunk;
  const long long stride = static_cast<long long>(gridDim.x) * kQWarps;
  const int group = layer / dm.rs_group;
  const uint8_t* map_g = cv.map + static_cast<long long>(group) * dm.batch * dm.max_chunks;
  const int32_t* slot_g = cv.slot + static_cast<long long>(group) * dm.batch * dm.max_chunks;

  const int32_t* count_g = cv.count + static_cast<long long>(group) * dm.batch * 4;
  auto tile_ref = [&](long long id) {
    // id = ((b * C + c) * tpc + j) * H + h : heads fastest, so neighbouring warps read
    // neighbouring 256-byte segments of the same token rows
    TileRef r;
    r.h = static_cast<int>(id % H);
    long long x = id / H;
    r.j = static_cast<int>(x % tpc);
    x /= tpc;
    if (!flush) {
      const int c = static_cast<int>(x % C);
      r.b = static_cast<int>(x / C);
      r.x = r.h * kHeadDim;
      r.y = r.b * T + c * dm.chunk + r.j * kTileTokens;
      const long long tbl = static_cast<long long>(r.b) * dm.max_chunks + c;
      r.w = map_g[tbl];                      // loaded one tile ahead of their use
      r.slot = slot_g[tbl];
    } else {
      // flush of a full tail: the source is the tail itself ([layer][b][h][row][128]); the target is
      // the sequence's newest chunk, marked with bit 7 in the map while its rows are being packed
      r.b = static_cast<int>(x);
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
  TileRef cur = tile_ref(id);
  fetch(&mapK, cur, bufK, barK);
  fetch(&mapV, cur, bufV, barV);
  uint32_t parity = 0;
  bool store_pending = false;
  int failed = 0;                             // 1: key rows never arrived, 2: value rows

  for (; id < n_tiles; id += stride) {
    const long long next = id + stride;
    TileRef nxt = cur;
    if (next < n_tiles) nxt = tile_ref(next);
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
        copy_raw_rows(bufK, tile, lane);
      } else {
        if (store_pending) {                  // the previous tile's bulk store must have read `out`
          if (lane == 0) bulk_store_wait_read();
          __syncwarp();
          store_pending = false;
        }
        if (w == 0) encode_keys<2, BF16>(bufK, out, lane);
        else if (w == 1) encode_keys<4, BF16>(bufK, out, lane);
        else encode_keys<8, BF16>(bufK, out, lane);
      }
    }
    __syncwarp();                             // every lane is done reading bufK
    if (next < n_tiles) fetch(&mapK, nxt, bufK, barK);

    // ---- values
    if (!mbar_wait_bounded(barV, parity)) { failed = 2; break; }
    if (valid) {
      if (w == 3) {
        copy_raw_rows(bufV, tile + 8192, lane);
      } else {
        if (w == 0) encode_values<2, BF16>(bufV, out, prm, lane);
        else if (w == 1) encode_values<4, BF16>(bufV, out, prm, lane);
        else encode_values<8, BF16>(bufV, out, prm, lane);
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

// cuTensorMapEncodeTiled through the runtime's driver entry-point lookup (no link against libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

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

cudaError_t launch_quantize(const Dims& dm, const CacheView& cv, const void* K, const void* V, int T,
                            int layer, cudaStream_t st) {
  const int C = T / dm.chunk;
  const long long n_tiles = static_cast<long long>(dm.batch) * C * (dm.chunk / kTileTokens) * dm.n_kv_heads;
  if (n_tiles > 0) {
    CUtensorMap mapK, mapV;
    const long long rows = static_cast<long long>(dm.batch) * T, cols = static_cast<long long>(dm.n_kv_heads) * kHeadDim;
    if (!make_tile_map(&mapK, K, rows, cols) || !make_tile_map(&mapV, V, rows, cols)) return cudaErrorNotSupported;
    const size_t smem = static_cast<size_t>(kQWarps) * kWarpSmem + kQWarps * 16;
    const long long want = (n_tiles + kQWarps - 1) / kQWarps;
    const long long cap = 2ll * sm_count();                    // two resident CTAs per SM, grid-stride
    const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
    cudaError_t e;
    if (dm.dtype == MOQAE_DTYPE_BF16) {
      e = cudaFuncSetAttribute(quantize_pack_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      quantize_pack_kernel<true><<<grid, kQWarps * 32, smem, st>>>(dm, cv, mapK, mapV, T, layer, n_tiles, 0);
    } else {
      e = cudaFuncSetAttribute(quantize_pack_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      quantize_pack_kernel<false><<<grid, kQWarps * 32, smem, st>>>(dm, cv, mapK, mapV, T, layer, n_tiles, 0);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  dim3 g(8, dm.batch);
  tail_copy_kernel<<<g, 256, 0, st>>>(dm, cv, static_cast<const uint16_t*>(K), static_cast<const uint16_t*>(V), T, layer);
  return cudaGetLastError();
}

// Pack the full tails of `layer` into the chunk that launch_flush_route has just added to the tables.
cudaError_t launch_flush_quantize(const Dims& dm, const CacheView& cv, int layer, cudaStream_t st) {
  const long long n_tiles = static_cast<long long>(dm.batch) * (dm.chunk / kTileTokens) * dm.n_kv_heads;
  CUtensorMap mapK, mapV;
  const long long rows = static_cast<long long>(dm.n_layers) * dm.batch * dm.n_kv_heads * dm.tail_capacity;
  if (!make_tile_map(&mapK, cv.tail_k, rows, kHeadDim) || !make_tile_map(&mapV, cv.tail_v, rows, kHeadDim))
    return cudaErrorNotSupported;
  const size_t smem = static_cast<size_t>(kQWarps) * kWarpSmem + kQWarps * 16;
  const long long want = (n_tiles + kQWarps - 1) / kQWarps;
  const long long cap = 2ll * sm_count();
  const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
  cudaError_t e;
  if (dm.dtype == MOQAE_DTYPE_BF16) {
    e = cudaFuncSetAttribute(quantize_pack_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    quantize_pack_kernel<true><<<grid, kQWarps * 32, smem, st>>>(dm, cv, mapK, mapV, 0, layer, n_tiles, 1);
  } else {
    e = cudaFuncSetAttribute(quantize_pack_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    quantize_pack_kernel<false><<<grid, kQWarps * 32, smem, st>>>(dm, cv, mapK, mapV, 0, layer, n_tiles, 1);
  }
  return cudaGetLastError();
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
