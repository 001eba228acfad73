// The quantiser of one 32-token tile as warp-level device code: group statistics, scale / zero,
// codes, bit-packing into the storage order of the decode lanes.  Used by the kernel that
// quantises K/V rows from memory and by the projection kernel that quantises them out of its
// accumulators; both feed it 32 rows of 256 bytes in shared memory.
#pragma once

#include "common.cuh"

namespace moqae {

namespace {

constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23

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
// `out` is the start of the tile image (metadata at its documented offsets); `pay_at`, if given,
// is where the key payload goes instead of out + 1024 (a warp that assembles only the key part
// of a tile keeps metadata and payload side by side).
// SHORT = false: all 32 rows are tokens (n_valid is ignored and the row tests fold away).
template <int BITS, bool BF16, bool SHORT = false>
__device__ __forceinline__ void encode_keys(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, int lane,
                                            int n_valid_arg = kTileTokens, uint8_t* pay_at = nullptr) {
  const int n_valid = SHORT ? n_valid_arg : kTileTokens;
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  const uint2* rows = reinterpret_cast<const uint2*>(in) + lane;         // row t at rows[32 * t]
  uint32_t mn01, mn23, mx01, mx23;
  {
    const uint2 w = rows[0];
    mn01 = mx01 = w.x; mn23 = mx23 = w.y;
  }
#pragma unroll
  for (int t = 1; t < kTileTokens; ++t) {
    // rows past n_valid are padding of a short chunk: the group is the chunk's own tokens
    const uint2 w = rows[t < n_valid ? 32 * t : 0];
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
  uint8_t* pay = pay_at ? pay_at : out + kMetaBytes;
  const uint64_t negz01 = pack_f2(-zf[0], -zf[1]), negz23 = pack_f2(-zf[2], -zf[3]);
  const uint64_t inv01 = pack_f2(inv[0], inv[1]), inv23 = pack_f2(inv[2], inv[3]);
  const int q = lane >> 3, l7 = lane & 7;
#pragma unroll
  for (int t = 0; t < kTileTokens; ++t) {
    const uint2 w = rows[32 * t];
    uint32_t u0, u1, u2, u3;
    encode2<BF16>(w.x, negz01, inv01, u0, u1);
    encode2<BF16>(w.y, negz23, inv23, u2, u3);
    uint32_t p = pack4<BITS>(u0, u1, u2, u3);
    if (t >= n_valid) p = 0u;                  // padding positions carry code 0
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
template <int BITS, bool BF16, bool SHORT = false>
__device__ __forceinline__ void encode_values(const uint8_t* __restrict__ in, uint8_t* __restrict__ out,
                                              float4* __restrict__ prm, int lane, int n_valid_arg = kTileTokens,
                                              uint8_t* pay_at = nullptr) {
  const int n_valid = SHORT ? n_valid_arg : kTileTokens;
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  uint16_t* meta = reinterpret_cast<uint16_t*>(out);
  {
    // statistics: lane = token.  Its row is read in 16-byte units; within each half of the row
    // (two channel groups = 8 units) lane t starts at unit t & 7, so the 32 lanes of one load
    // spread over all eight 16-byte bank groups (4 lanes each: the minimum for 512 bytes).
    const int t = lane;
    const uint4* row = reinterpret_cast<const uint4*>(in + t * 256);
    const int blk = t >> 4, half = (t >> 3) & 1, t4 = (t >> 1) & 3, e = t & 1;
    constexpr uint32_t kPosInf = BF16 ? 0x7F807F80u : 0x7C007C00u, kNegInf = BF16 ? 0xFF80FF80u : 0xFC00FC00u;
    uint32_t mn4[4], mx4[4];
#pragma unroll
    for (int cp = 0; cp < 2; ++cp) {
      uint32_t mnA = kPosInf, mxA = kNegInf, mnB = kPosInf, mxB = kNegInf;     // A: this lane's first group, B: its second
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int u = k ^ (t & 7);
        const uint4 v = row[8 * cp + u];
        const uint32_t a = min2<BF16>(min2<BF16>(v.x, v.y), min2<BF16>(v.z, v.w));
        const uint32_t b = max2<BF16>(max2<BF16>(v.x, v.y), max2<BF16>(v.z, v.w));
        // units 0..3 belong to group 2cp, 4..7 to 2cp + 1; u >> 2 = (k >> 2) ^ ((t >> 2) & 1), so the
        // first four loads of a lane fall into one group and the last four into the other
        if (k < 4) { mnA = min2<BF16>(mnA, a); mxA = max2<BF16>(mxA, b); }
        else { mnB = min2<BF16>(mnB, a); mxB = max2<BF16>(mxB, b); }
      }
      const bool swap = (t >> 2) & 1;          // lanes with bit 2 set met group 2cp + 1 first
      mn4[2 * cp] = swap ? mnB : mnA; mx4[2 * cp] = swap ? mxB : mxA;
      mn4[2 * cp + 1] = swap ? mnA : mnB; mx4[2 * cp + 1] = swap ? mxA : mxB;
    }
#pragma unroll
    for (int cg = 0; cg < 4; ++cg) {
      const uint32_t mn = mn4[cg], mx = mx4[cg];
      float zf, inv;
      uint16_t sb, zb;
      group_params(fminf(lo_f<BF16>(mn), hi_f<BF16>(mn)), fmaxf(lo_f<BF16>(mx), hi_f<BF16>(mx)), qmax, sb, zb, zf, inv);
      if (t >= n_valid) {                      // padding token: scale 0, zero 0, every code 0
        sb = 0; zb = 0; zf = 0.0f; inv = 0.0f;
      }
      // [token][group], the four groups of a token rotated by t / 2: the 32 lanes of this store spread evenly
      // over the eight 16-byte bank groups, and the four entries of one token that the encode pass reads in
      // one load sit in one 64-byte row
      prm[4 * t + ((cg + (t >> 1)) & 3)] = make_float4(-zf, -zf, inv, inv);
      meta[256 + ((((blk * 2 + (cg >> 1)) * 4 + t4) * 4 + (cg & 1) * 2 + half) * 2) + e] = sb;
      meta[384 + ((((blk * 4 + cg) * 4 + t4) * 2 + half) * 2) + e] = zb;
    }
  }
  __syncwarp();
  // codes: lane = channels 4*lane .. 4*lane+3 (group p = lane / 8); one word set per 4 tokens
  const int p = lane >> 3, g = lane & 7;
  const uint2* rows = reinterpret_cast<const uint2*>(in) + lane;
  uint8_t* pay = pay_at ? pay_at : out + kMetaBytes + kTileTokens * 16 * BITS;
  // not unrolled over the two halves: the kernel's warps sit in different phases of different widths, and
  // keeping their code small enough for the instruction cache is worth more than the longer basic block
#pragma unroll 1
  for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
    for (int t4 = 0; t4 < 4; ++t4) {
      uint32_t u[4][4];                      // [byte position half + 2e][channel]
#pragma unroll
      for (int bp = 0; bp < 4; ++bp) {
        const int t = 16 * blk + 8 * (bp & 1) + 2 * t4 + (bp >> 1);
        const uint2 w = rows[32 * t];
        const ulonglong2 zi = *reinterpret_cast<const ulonglong2*>(prm + 4 * t + ((p + (t >> 1)) & 3));   // (-z, -z), (inv, inv)
        encode2<BF16>(w.x, zi.x, zi.y, u[bp][0], u[bp][1]);
        encode2<BF16>(w.y, zi.x, zi.y, u[bp][2], u[bp][3]);
        if (t >= n_valid) {                    // padding token: code 0 whatever the row holds
#pragma unroll
          for (int k = 0; k < 4; ++k) u[bp][k] = __float_as_uint(kMagic);
        }
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
template <bool SHORT = false>
__device__ __forceinline__ void copy_raw_rows(const uint8_t* __restrict__ in, uint8_t* __restrict__ dst, int lane,
                                              int n_valid_arg = kTileTokens) {
  const int n_valid = SHORT ? n_valid_arg : kTileTokens;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int idx = i * 32 + lane;
    const int row = idx >> 4, U = idx & 15;
    const int up = (U & 8) | ((U ^ row) & 7);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);      // rows past a short chunk's tokens are zero
    if (row < n_valid) v = *reinterpret_cast<const uint4*>(in + row * 256 + U * 16);
    *reinterpret_cast<uint4*>(dst + row * 256 + up * 16) = v;
  }
}

}  // namespace

}  // namespace moqae
