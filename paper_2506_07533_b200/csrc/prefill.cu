// Causal prefill attention over the quantised chunks (Section 3.1: a block quantises its
// chunks and then proceeds with its attention; Limitations section: keys are dequantised to
// 16-bit floats before the product with the query).
//
// A dense contraction, so it runs on the 5th-generation tensor cores: one CTA owns 256
// consecutive query positions (two tiles of 128) of one query head and walks the cache in
// blocks of 128 tokens (four storage tiles, in token order through the chunk map).  Per block
//   K^, V^       fp16 operand tiles [128 tokens x 128 channels] in shared memory, two stages.
//                Without a workspace eight warps expand the packed tiles of the block (core-matrix
//                layout without swizzle); with one, prefill_dequant_kernel has expanded the whole
//                layer into fp16 rows beforehand and two threads fetch the block with tiled TMA
//                copies into the 128-byte swizzled layout;
//   S_i = Q_i K^T  8 x tcgen05.mma (M 128, N 128, K 16) per query tile, fp32 in tensor memory;
//   softmax      one thread per query row (two with a workspace, 64 columns each) reads S_i with
//                tcgen05.ld, applies the causal mask, keeps a lazily moved reference maximum and
//                the running sum, and writes P_i as packed fp16 over the consumed columns of S_i;
//   O_i += P_i V^  8 x tcgen05.mma with P_i as a tensor-memory operand, accumulating in tensor
//                memory across blocks (rescaled in place on the rare blocks where the reference
//                maximum moves).
// The roles run concurrently and meet on mbarriers (plus one named barrier per pair of softmax
// warps that share rows).  Every mbarrier wait is bounded; on expiry the CTA records
// MOQAE_ERR_TIMEOUT, every role stops and the tensor memory is still freed.
#include <cstring>

#include <cuda_bf16.h>

#include "ptx.cuh"

namespace moqae {

namespace {

constexpr int kQTile = 128;                    // query rows per CTA
constexpr int kKvBlock = 128;                  // tokens per block (four storage tiles)
constexpr long long kPrefillWaitCycles = 1ll << 31;    // about a second: no wait of a healthy launch comes near

// ---- tcgen05 wrappers -------------------------------------------------------------------
// Shared-memory matrix descriptor, no swizzle: start address, leading-dimension byte offset
// (between the two 8-element halves of a K step, or between groups of 8 K rows for an
// MN-major operand) and stride byte offset (between groups of 8 rows / of 8 MN elements), all
// in units of 16 bytes; bits 46..47 = 1 is the descriptor version of this architecture.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((saddr >> 4) & 0x3fffu) | (static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fffu) << 16) |
         (static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46);
}
// Instruction descriptor of kind::f16: fp32 accumulator, fp16 A and B, M = 128, N = 128;
// bit 16 set = B is MN-major (its N index is the contiguous one).
constexpr uint32_t kIdescS = (1u << 4) | (16u << 17) | (8u << 24);
constexpr uint32_t kIdescPV = kIdescS | (1u << 16);

// D (tensor memory) = / += A B with the A operand read from tensor memory: row = lane, 16-bit
// elements packed two per 32-bit column (element 2j in the low half of column j), 8 columns per
// K step of 16.  The B descriptor arrives as its two words so that the issuing thread only adds
// a block offset to the low one (start address field; it never carries out of its 14 bits).
__device__ __forceinline__ void umma_f16_ta(uint32_t tmem_d, uint32_t tmem_a, uint32_t bdesc_lo, uint32_t bdesc_hi, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\n.reg .b64 bd;\nsetp.ne.b32 p, %5, 0;\nmov.b64 bd, {%2, %3};\n"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n}\n"
               ::"r"(tmem_d), "r"(tmem_a), "r"(bdesc_lo), "r"(bdesc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// The same with both operands in shared memory.
__device__ __forceinline__ void umma_f16_ss(uint32_t tmem_d, uint32_t adesc_lo, uint32_t adesc_hi, uint32_t bdesc_lo, uint32_t bdesc_hi,
                                            uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\n.reg .b64 ad, bd;\nsetp.ne.b32 p, %6, 0;\nmov.b64 ad, {%1, %2};\nmov.b64 bd, {%3, %4};\n"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n}\n"
               ::"r"(tmem_d), "r"(adesc_lo), "r"(adesc_hi), "r"(bdesc_lo), "r"(bdesc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld32(float (&v)[32], uint32_t taddr) {
  uint32_t r[32];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// ---- operand tiles in shared memory -------------------------------------------------------
// K-major operand (Q; K^ with the 128 token rows of a block): element (row n, k) of a
// ROWS x 128 fp16 tile.  Core matrix = 8 rows x 8 elements (128 bytes); the ROWS/8 core matrices
// of one 8-element K slab are contiguous (128 B between row groups), K slabs follow each other.
template <int ROWS>
__device__ __forceinline__ int kmajor_unit_offset(int n, int k8) {       // byte offset of the 16-byte unit (n, k8*8..+7)
  return (k8 * (ROWS / 8) + (n >> 3)) * 128 + (n & 7) * 16;
}
// MN-major operand (V^: rows = tokens (K of the MMA), contiguous index = channels): core
// matrix = 8 tokens x 8 channels; the 16 channel groups of one 8-token slab are contiguous.
__device__ __forceinline__ int mnmajor_unit_offset(int t, int c8) {      // byte offset of the 16-byte unit (t, c8*8..+7)
  return ((t >> 3) * 16 + c8) * 128 + (t & 7) * 16;
}

// Where the dequantising code puts the 16-byte unit (token row t of the block, channels
// 8 c8 .. 8 c8 + 7): into the operand tile in shared memory, or (ROWS = true) into plain rows of
// 256 bytes in global memory.
template <bool ROWS, bool IS_V> __device__ __forceinline__ int dst_unit_offset(int t, int c8) {
  return ROWS ? t * 256 + c8 * 16 : (IS_V ? mnmajor_unit_offset(t, c8) : kmajor_unit_offset<128>(t, c8));
}

__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// eight 16-bit inputs (one uint4) -> eight fp16
template <bool BF16> __device__ __forceinline__ uint4 to_fp16x8(uint4 v) {
  if (!BF16) return v;
  uint4 o;
  o.x = pack_h2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u));
  o.y = pack_h2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
  o.z = pack_h2(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u));
  o.w = pack_h2(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
  return o;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(r) : "f"(x));
  return r;
}
// packed fp32 pairs: one instruction for two lanes of arithmetic
__device__ __forceinline__ uint64_t pack_f2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack_f2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;\n" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ---- dequantisation of one 32-token storage tile into the operand tiles --------------------
// The packed layout is the one the decode kernel's lanes consume (lane = 4g + t4); the same
// 16-byte units are read here, straight from global memory, and expanded to fp16.
template <int BITS> __host__ __device__ constexpr int key_reg_channel_lo(int r) {
  constexpr int n = 32 / BITS;
  return (r / (n / 2)) * n + ((r % (n / 2)) / (n / 4)) * (n / 4) + r % (n / 4);
}

// Two codes that sit at the same bit position `pos` of the two half-words of `w` -> (code_lo,
// code_hi) as fp16: shifting them to bit 0 and OR-ing 0x6400 gives 1024 + code exactly.
template <int BITS> __device__ __forceinline__ uint32_t codes_to_half2(uint32_t w, int pos) {
  constexpr uint32_t mask = ((1u << BITS) - 1u) * 0x00010001u;
  uint32_t x = ((w >> pos) & mask) | 0x64006400u, r;
  asm("sub.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(x), "r"(0x64006400u));
  return r;
}
__device__ __forceinline__ uint32_t hfma2_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.f16x2 %0, %1, %2, %3;\n" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

// Keys.  A payload word masked at one code position carries the codes of channels c and
// c + n/2 (n = codes per word); the scale and zero arrays hold exactly those pairs, so one
// packed FMA dequantises two channels: K^ = RN(code * scale + zero) in fp16.
template <int BITS, bool ROWS>
__device__ __forceinline__ void dequant_keys(const uint8_t* __restrict__ tile, uint8_t* sK, int sub, int lane) {
  constexpr int n = 32 / BITS, regs = n / 2, direct = n / 4;
  const int g = lane >> 2, t4 = lane & 3;
  uint32_t sc[16], zr[16];                 // register r: (lo, hi) = channels cl(r), cl(r) + n/2 of quarter t4
  {
    const uint4* sp = reinterpret_cast<const uint4*>(tile) + t4;
    const uint4* zp = reinterpret_cast<const uint4*>(tile + 256) + t4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint4 s4 = __ldg(sp + 4 * i), z4 = __ldg(zp + 4 * i);
      sc[4 * i] = s4.x; sc[4 * i + 1] = s4.y; sc[4 * i + 2] = s4.z; sc[4 * i + 3] = s4.w;
      zr[4 * i] = z4.x; zr[4 * i + 1] = z4.z; zr[4 * i + 2] = z4.y; zr[4 * i + 3] = z4.w;   // stored in order 0, 2, 1, 3
    }
  }
  const uint8_t* kpay = tile + kMetaBytes;
#pragma unroll 1
  for (int blk = 0; blk < 2; ++blk)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      uint32_t w[BITS];
      if (BITS == 2) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(kpay + (blk * 32 + lane) * 16));
        w[0] = hh ? v.z : v.x; w[1] = hh ? v.w : v.y;
      } else if (BITS == 4) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(kpay + ((2 * blk + hh) * 32 + lane) * 16));
        w[0] = v.x; w[1] = v.y; w[2 % BITS] = v.z; w[3 % BITS] = v.w;
      } else {
#pragma unroll
        for (int j2 = 0; j2 < 2; ++j2) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(kpay + (((2 * blk + hh) * 2 + j2) * 32 + lane) * 16));
          w[(4 * j2) % BITS] = v.x; w[(4 * j2 + 1) % BITS] = v.y; w[(4 * j2 + 2) % BITS] = v.z; w[(4 * j2 + 3) % BITS] = v.w;
        }
      }
      // value pair of register r: channels (cl, cl + n/2); val[c] collects them by channel pair
      uint32_t byreg[16];
#pragma unroll
      for (int r = 0; r < 16; ++r) {
        const int j = r / regs, s = (r % regs) / direct, m = r % direct;
        byreg[r] = hfma2_u32(codes_to_half2<BITS>(w[j], 8 * s + BITS * m), sc[r], zr[r]);
      }
      // channels cc and cc + 1 (cc even) of the piece: low or high halves of two neighbouring registers
      const int row = 32 * sub + 16 * blk + 8 * hh + g;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        uint32_t o[4];
#pragma unroll
        for (int e2 = 0; e2 < 4; ++e2) {
          const int cc = 8 * u + 2 * e2;                      // even channel of the pair
          const int j = cc / n, i = cc % n;                   // word, position inside the word
          const bool hi = i >= n / 2;
          const int i2 = i % (n / 2);
          const int ra = j * regs + (i2 / direct) * direct + i2 % direct;         // register of channel cc
          const int i3 = (i + 1) % (n / 2);
          const int rb = j * regs + (i3 / direct) * direct + i3 % direct;         // register of channel cc + 1
          o[e2] = __byte_perm(byreg[ra], byreg[rb], hi ? 0x7632 : 0x5410);
        }
        *reinterpret_cast<uint4*>(sK + dst_unit_offset<ROWS, false>(row, 4 * t4 + u)) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
}

// Values.  A payload word masked at one slot carries the codes of tokens e = 0, 1 of one
// channel row; the scale and zero arrays hold those token pairs per channel group.
template <int BITS, bool ROWS>
__device__ __forceinline__ void dequant_values(const uint8_t* __restrict__ tile, uint8_t* sV, int sub, int lane) {
  constexpr int per = 8 / BITS;                                   // channel rows per word
  const int g = lane >> 2, t4 = lane & 3;
  const uint8_t* vpay = tile + kMetaBytes + kTileTokens * 16 * BITS;
#pragma unroll 1
  for (int blk = 0; blk < 2; ++blk) {
    uint32_t sw[4][2], zw[4][2];                                  // [channel group][half]: fp16 pair (e = 0, 1)
#pragma unroll
    for (int cp = 0; cp < 2; ++cp) {
      const uint4 s4 = __ldg(reinterpret_cast<const uint4*>(tile + 512 + ((blk * 2 + cp) * 4 + t4) * 16));
      sw[2 * cp][0] = s4.x; sw[2 * cp][1] = s4.y; sw[2 * cp + 1][0] = s4.z; sw[2 * cp + 1][1] = s4.w;
    }
#pragma unroll
    for (int cg = 0; cg < 4; ++cg) {
      const uint2 z2 = __ldg(reinterpret_cast<const uint2*>(tile + 768 + ((blk * 4 + cg) * 4 + t4) * 8));
      zw[cg][0] = z2.x; zw[cg][1] = z2.y;
    }
    uint32_t wv[2 * BITS];
#pragma unroll
    for (int u = 0; u < BITS / 2; ++u) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(vpay + ((blk * (BITS / 2) + u) * 32 + lane) * 16));
      wv[4 * u] = v.x; wv[4 * u + 1] = v.y; wv[4 * u + 2] = v.z; wv[4 * u + 3] = v.w;
    }
#pragma unroll
    for (int cg = 0; cg < 4; ++cg)
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t v[4];                                             // channel rows r4 = 0..3: (token e = 0, token e = 1)
#pragma unroll
        for (int r4 = 0; r4 < 4; ++r4) {
          const int R = 4 * cg + r4;
          v[r4] = hfma2_u32(codes_to_half2<BITS>(wv[R / per], BITS * (R % per) + 8 * half), sw[cg][half], zw[cg][half]);
        }
        const int tok = 32 * sub + 16 * blk + 8 * half + 2 * t4;
        // channels 32cg + 4g .. +3: half of the 16-byte unit c8 = 4cg + g/2, one store per token
        *reinterpret_cast<uint2*>(sV + dst_unit_offset<ROWS, true>(tok, 4 * cg + (g >> 1)) + (g & 1) * 8) =
            make_uint2(__byte_perm(v[0], v[1], 0x5410), __byte_perm(v[2], v[3], 0x5410));
        *reinterpret_cast<uint2*>(sV + dst_unit_offset<ROWS, true>(tok + 1, 4 * cg + (g >> 1)) + (g & 1) * 8) =
            make_uint2(__byte_perm(v[0], v[1], 0x7632), __byte_perm(v[2], v[3], 0x7632));
      }
  }
}

// 32 rows of 256 bytes in the input dtype -> one operand tile.  SWIZZLED: rows of a 16-bit
// pool tile (units permuted inside each row); otherwise plain rows (the tail), of which only
// the first n_valid exist.
template <bool BF16, bool SWIZZLED, bool IS_V, bool ROWS>
__device__ __forceinline__ void copy_rows(const uint8_t* __restrict__ src, uint8_t* dst, int sub, int n_valid, int lane) {
#pragma unroll 4
  for (int i = 0; i < 16; ++i) {
    const int idx = i * 32 + lane;
    const int row = idx >> 4, U = idx & 15;
    const int up = SWIZZLED ? ((U & 8) | ((U ^ row) & 7)) : U;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < n_valid) v = to_fp16x8<BF16>(__ldg(reinterpret_cast<const uint4*>(src + row * 256 + up * 16)));
    const int off = dst_unit_offset<ROWS, IS_V>(32 * sub + row, U);
    *reinterpret_cast<uint4*>(dst + off) = v;
  }
}

// ---- the kernel ----------------------------------------------------------------------------
// Roles without a workspace (17 warps): warps 0..3 and 4..7 are the softmax threads of the CTA's
// two query tiles (one row each, tensor-memory lane = tid % 128); warps 8..11 dequantise the
// keys and warps 12..15 the values of every block (one storage tile each); warp 16 issues the
// MMAs.  With a workspace (19 warps): warps 8..15 are a second set of softmax threads (warp w + 8
// shares the rows of warp w and takes the other 64 columns), warps 17 and 18 fetch K^ and V^.  Shared
// memory holds the two query tiles and kStages blocks of K^ and of V^; the probabilities are an
// A operand read from tensor memory.  Tensor memory (512 columns):
//   S_i   128 columns at 128 i        scores (fp32) of the current block; P_i (packed fp16, 64
//                                     columns) overwrites its first half chunk by chunk as the
//                                     scores are read
//   O_i   128 columns at 256 + 128 i
// Every product is M 128 x N 128 x K 16, the shape at which the tensor pipe runs at its peak
// when fed by one issuing thread.  The two tiles alternate: while the softmax threads of one
// work on S_i, the pipe runs O += P V^ and the next S of the other.  The roles meet only on
// mbarriers:
//   kfull[st] / vfull[st]   K^ / V^ of a block are in stage st               (4 dequant warps, or the TMA bytes)
//   kfree[st] / vfree[st]   the products that read stage st are done         (tcgen05.commit)
//   sfull[i]                S_i = Q_i K^T is in tensor memory                (tcgen05.commit)
//   pfull[i]                P_i is in tensor memory                          (the tile's 4 or 8 softmax warps)
//   ofull[i]                the last O_i += P_i V^ is done                   (tcgen05.commit, once)
// Stage barriers complete once per kStages blocks, tile barriers once per block, and every
// waiter follows its barrier completion by completion, so waiting on the parity of the
// completion index is exact.  The MMAs of one thread execute in issue order: S_i of block
// kb + 1 is issued after O_i += P_i V^ of block kb, so it may overwrite P_i, and its completion
// tells the softmax threads that O_i is at rest (they rescale it in place when the reference
// maximum moves).
constexpr int kSoftmaxWarps = 8, kDequantWarps = 8;   // dequant: 4 warps for keys, 4 for values
// Without a workspace: 8 softmax + 8 dequantise + 1 issue warp.  With one: 16 softmax warps (two
// per 32 rows, each taking half of a block's columns), the issue warp and two fetch warps.
__host__ __device__ constexpr int block_threads(bool pre) { return (kSoftmaxWarps + kDequantWarps + (pre ? 3 : 1)) * 32; }
constexpr int kIssueWarp = kSoftmaxWarps + kDequantWarps;
constexpr int kExchangeBytes = 256 * 2 * 4 + 2 * 8 * 2 * 4;   // per row and half: one float; per block parity, pair, half: one flag
constexpr int kTmemCols2 = 512;
constexpr float kSumLimit = 16384.0f;          // a chunk whose weights sum to less cannot overflow fp16 (65504)
constexpr int kStages = 2;
constexpr int kStageBytes = kKvBlock * 128 * 2;  // one K^ / V^ stage
constexpr int kQTileBytes = kQTile * 128 * 2;

enum { BAR_KFULL = 0, BAR_VFULL = kStages, BAR_KFREE = 2 * kStages, BAR_VFREE = 3 * kStages,
       BAR_SFULL = 4 * kStages, BAR_PFULL = 4 * kStages + 2, BAR_OFULL = 4 * kStages + 4, BAR_COUNT = 4 * kStages + 6 };

// 32 consecutive 32-bit columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_st32u(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
               "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
               "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
               ::"r"(taddr),
                 "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                 "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
                 "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
                 "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
               : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  uint32_t r[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i]);
  tmem_st32u(taddr, r);
}

// 16 consecutive 32-bit columns; the store is not waited for here (tmem_st_wait)
__device__ __forceinline__ void tmem_st16u_nowait(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
               "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n"
               ::"r"(taddr),
                 "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                 "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16u(uint32_t (&r)[16], uint32_t taddr) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

// Where the cache of one (layer, sequence, kv head) lives, and how to reach a 32-token tile of it.
struct KvSource {
  const CacheView* cv;
  const Dims* dm;
  long long tbl, tail_base;
  int layer, b, h, chunk_tokens, tail_len, tpc;
};

__device__ __forceinline__ KvSource kv_source(const CacheView& cv, const Dims& dm, int layer, int b, int h) {
  KvSource ks;
  ks.cv = &cv; ks.dm = &dm; ks.layer = layer; ks.b = b; ks.h = h;
  const int group = layer / dm.rs_group;
  ks.tbl = (static_cast<long long>(group) * dm.batch + b) * dm.max_chunks;
  const int32_t* cnt = cv.count + (static_cast<long long>(group) * dm.batch + b) * 4;
  ks.chunk_tokens = min(cnt[0] + cnt[1] + cnt[2] + cnt[3], dm.max_chunks) * dm.chunk;
  ks.tail_len = min(cv.tail_len[layer * dm.batch + b], dm.tail_capacity);
  ks.tpc = dm.chunk / kTileTokens;
  ks.tail_base = ((static_cast<long long>(layer) * dm.batch + b) * dm.n_kv_heads + h) * dm.tail_capacity;
  return ks;
}

template <bool BF16, bool ROWS>
__device__ __forceinline__ void dequant_subtile(const KvSource& ks, int pos0, int sub, bool is_v, uint8_t* dst, int lane) {
  const CacheView& cv = *ks.cv;
  const Dims& dm = *ks.dm;
  if (pos0 < ks.chunk_tokens) {
    const int c = pos0 / dm.chunk, j = (pos0 % dm.chunk) / kTileTokens;
    const int w = cv.map[ks.tbl + c] & 3;
    const long long slot = cv.slot[ks.tbl + c];
    long long cap = 0;
    const uint8_t* pool = nullptr;
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (w == k) { cap = cv.capacity[k]; pool = cv.pool[k]; }
    const long long tb = tile_bytes_of_expert(w);
    const long long s = slot < 0 ? 0 : (slot < cap ? slot : cap - 1);          // never leave the pool
    const uint8_t* tile = pool + ((((static_cast<long long>(ks.layer) * dm.batch + ks.b) * dm.n_kv_heads + ks.h) * cap + s) * ks.tpc + j) * tb;
    if (w == 0) { if (is_v) dequant_values<2, ROWS>(tile, dst, sub, lane); else dequant_keys<2, ROWS>(tile, dst, sub, lane); }
    else if (w == 1) { if (is_v) dequant_values<4, ROWS>(tile, dst, sub, lane); else dequant_keys<4, ROWS>(tile, dst, sub, lane); }
    else if (w == 2) { if (is_v) dequant_values<8, ROWS>(tile, dst, sub, lane); else dequant_keys<8, ROWS>(tile, dst, sub, lane); }
    else if (is_v) copy_rows<BF16, true, true, ROWS>(tile + 8192, dst, sub, 32, lane);
    else copy_rows<BF16, true, false, ROWS>(tile, dst, sub, 32, lane);
  } else {
    const int ti0 = pos0 - ks.chunk_tokens;
    const int n_valid = max(0, min(32, ks.tail_len - ti0));
    const uint8_t* src = reinterpret_cast<const uint8_t*>(is_v ? cv.tail_v : cv.tail_k) + (ks.tail_base + ti0) * 256;
    if (is_v) copy_rows<BF16, false, true, ROWS>(src, dst, sub, n_valid, lane);
    else copy_rows<BF16, false, false, ROWS>(src, dst, sub, n_valid, lane);
  }
}

// ---- dequantise once: the cache of one layer as fp16 rows -----------------------------------
// K^ and V^ of (sequence b, kv head h) as [t_pad][128] fp16 rows in a caller-provided scratch,
// t_pad = the prompt length rounded up to whole blocks; rows past the cached tokens are zero.
// One CTA per 32-token storage tile: warp 0 expands the keys, warp 1 the values.  With this
// pass in front, the attention kernel below fetches ready-made operand tiles with TMA instead of
// expanding every tile again in each of the T / 256 CTAs that walk over it.
template <bool BF16>
__global__ void __launch_bounds__(64) prefill_dequant_kernel(Dims dm, CacheView cv, int layer, int t_pad, uint8_t* __restrict__ kd,
                                                             uint8_t* __restrict__ vd) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pos0 = blockIdx.x * kTileTokens, h = blockIdx.y, b = blockIdx.z;
  const KvSource ks = kv_source(cv, dm, layer, b, h);
  uint8_t* dst = (warp ? vd : kd) + ((static_cast<long long>(b) * dm.n_kv_heads + h) * t_pad + pos0) * 256;
  dequant_subtile<BF16, true>(ks, pos0, 0, warp != 0, dst, lane);
}

// Descriptors of the 128-byte swizzled layouts TMA writes (bits 61..63 = 2).  K-major (K^: one
// row of 64 channels = 128 bytes, 1 KiB between groups of 8 token rows; the leading offset is not
// used) and MN-major (V^: 64 channels contiguous, 128 bytes between the 8 tokens of a group,
// leading offset = distance between the two 64-channel halves, stride offset = 1 KiB between
// groups of 8 tokens).
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return make_desc(saddr, lbo_bytes, sbo_bytes) | (2ull << 61);
}

template <bool BF16, bool PRE>
__global__ void __launch_bounds__(block_threads(PRE), 1)
prefill_attn_kernel(Dims dm, CacheView cv, const uint16_t* __restrict__ Q, int T, int layer, float scale_log2,
                    float* __restrict__ out, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    int t_pad) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // swizzled tiles want 1 KiB alignment
  uint8_t* sQ = smem;                               // two query tiles
  uint8_t* sK = sQ + 2 * kQTileBytes;               // kStages blocks
  uint8_t* sV = sK + kStages * kStageBytes;         // kStages blocks
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(sV + kStages * kStageBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + BAR_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* exch = reinterpret_cast<float*>(bar_mem + BAR_COUNT + 2);      // [256 rows][2 halves]
  volatile int* pair_flag = reinterpret_cast<volatile int*>(exch + 512);  // [2 block parities][8 pairs][2 halves]
  const uint32_t bar0 = smem_u32(bar_mem);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int pair = gridDim.x - 1 - blockIdx.x;      // longest rows of blocks first
  const int hq = blockIdx.y, b = blockIdx.z;
  const int H = dm.n_kv_heads, Hq = dm.n_q_heads;
  const int h = hq / (Hq / H);
  // blocks that tile i can see: up to the one holding its last row's own position
  const int nb_all = (T + kKvBlock - 1) / kKvBlock;
  const int nb0 = min(2 * pair + 1, nb_all), nb1 = min(2 * pair + 2, nb_all);

  if (warp == kIssueWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols2) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < BAR_COUNT; ++i) {
      // kfull / vfull: four dequantising warps, or the one thread that starts the TMA copies
      const int count = i < BAR_KFREE ? (PRE ? 1 : 4) : ((i >= BAR_PFULL && i < BAR_OFULL) ? (PRE ? 8 : 4) : 1);
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar(i)), "r"(count) : "memory");
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  // the CTA's 2 x 128 query rows as A operands (rows past the prompt are zero)
  for (int i = tid; i < 2 * kQTile * 16; i += block_threads(PRE)) {
    const int row = i >> 4, U = i & 15;             // row 0..255
    const int pos = 2 * pair * kQTile + row;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (pos < T)
      v = to_fp16x8<BF16>(__ldg(reinterpret_cast<const uint4*>(Q + ((static_cast<long long>(b) * T + pos) * Hq + hq) * kHeadDim + 8 * U)));
    *reinterpret_cast<uint4*>(sQ + (row >> 7) * kQTileBytes + kmajor_unit_offset<128>(row & 127, U)) = v;
  }
  fence_async_proxy();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // bounded wait that also gives up when another role has given up
  auto wait = [&](int which, int completion) -> bool {
    const uint32_t a = bar(which), parity = static_cast<uint32_t>(completion) & 1u;
    if (mbar_try_wait(a, parity)) return true;
    const long long t0 = clock64();
    while (!*abort_flag) {
      if (mbar_try_wait(a, parity)) return true;
      if (clock64() - t0 > kPrefillWaitCycles) *abort_flag = 1;
    }
    return false;
  };

  if (PRE && warp < kIssueWarp) {
    // ================= softmax, two threads per query row =================
    // Warps w and w + 8 share the 32 rows (tensor-memory lanes) of tile i = (w & 7) >> 2: the first
    // takes columns 0..63 of every block, the second columns 64..127.  Both keep the same
    // reference maximum; they meet once per block on a named barrier of their 64 threads, which
    // also orders "every score has been read" before "P overwrites the first half of S".
    const int half = warp >> 3;                     // which 64 columns
    const int i = (warp & 7) >> 2;                  // query tile
    const int nb = i ? nb1 : nb0;
    const int row = 128 * i + 32 * (warp & 3) + lane;           // 0..255 in the CTA
    const int qpos = 2 * pair * kQTile + row;
    const int pair_id = warp & 7;                   // the two warps of these rows
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t s_addr = lane_addr + 128 * i + 64 * half;     // this thread's 64 score columns
    const uint32_t p_addr = lane_addr + 128 * i + 32 * half;     // where its 32 packed columns of P go
    const uint32_t o_addr = lane_addr + 256 + 128 * i + 64 * half;   // the half of O it rescales and writes out
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;\n" ::"r"(1 + pair_id) : "memory"); };
    float m_ref = -INFINITY, l = 0.0f;
    bool ok = true;
    for (int kb = 0; kb < nb && ok; ++kb) {
      ok = __all_sync(0xffffffffu, wait(BAR_SFULL + i, kb));
      // a warp whose wait ran out still meets its partner on the pair barrier (which has no time
      // limit of its own) and tells it, so that both leave the loop after the same block
      if (ok) tc_fence_after();
      const bool diag = kb >= 2 * pair + i;
      const int rel = qpos - kb * kKvBlock - 64 * half;          // local columns 0..rel are visible
      uint32_t pk[32];
      float csum = 0.0f;
      // weights of this thread's 64 columns against m_ref; with want_max also their largest score
      auto weights = [&](bool want_max, float& mx) {
        csum = 0.0f;
        mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float v[32];
          tmem_ld32(v, s_addr + 32 * c);
          if (diag) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (32 * c + e > rel) v[e] = -INFINITY;
          }
          if (want_max) {
#pragma unroll
            for (int e = 0; e < 32; ++e) mx = fmaxf(mx, v[e]);
          }
          const uint64_t scale2 = pack_f2(scale_log2, scale_log2), negm2 = pack_f2(-m_ref, -m_ref);
          uint64_t part[2] = {0ull, 0ull};
#pragma unroll
          for (int e2 = 0; e2 < 16; ++e2) {
            float x0, x1;
            unpack_f2(fma_f2(pack_f2(v[2 * e2], v[2 * e2 + 1]), scale2, negm2), x0, x1);
            const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
            part[e2 & 1] = add_f2(part[e2 & 1], pack_f2(p0, p1));
            pk[16 * c + e2] = pack_h2(p0, p1);
          }
          float s0, s1;
          unpack_f2(add_f2(part[0], part[1]), s0, s1);
          csum += s0 + s1;
        }
      };
      float mx;
      if (ok) weights(false, mx);
      const bool over = ok && __any_sync(0xffffffffu, !(csum < kSumLimit));
      if (lane == 0) pair_flag[((kb & 1) * 8 + pair_id) * 2 + half] = (over ? 1 : 0) | (ok ? 0 : 2);
      pair_sync();                                   // both halves of S have been read; flags are visible
      const int flags = pair_flag[((kb & 1) * 8 + pair_id) * 2] | pair_flag[((kb & 1) * 8 + pair_id) * 2 + 1];
      if (flags & 2) {
        ok = false;
        break;
      }
      if (flags & 1) {
        // Rare (always on the first block): move the reference to the row's largest score of this
        // block and rescale what was accumulated against the old one.  O_i is at rest: S_i of this
        // block was issued after the last O_i += P_i V^.
        weights(true, mx);
        exch[row * 2 + half] = mx * scale_log2;      // scale_log2 > 0
        pair_sync();
        const float m_new = fmaxf(m_ref, ceilf(fmaxf(exch[row * 2], exch[row * 2 + 1])));
        const float corr = (m_ref == -INFINITY) ? 0.0f : ex2_approx(m_ref - m_new);
        if (kb > 0) {
#pragma unroll 1
          for (int o4 = 0; o4 < 2; ++o4) {
            float o[32];
            tmem_ld32(o, o_addr + 32 * o4);
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] *= corr;
            tmem_st32(o_addr + 32 * o4, o);
          }
        }
        l *= corr;
        m_ref = m_new;
        weights(false, mx);
        pair_sync();                                 // the partner has read its scores again, too
      }
      l += csum;
      tmem_st32u(p_addr, pk);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_PFULL + i));
    }
    if (ok && nb > 0) ok = __all_sync(0xffffffffu, wait(BAR_OFULL + i, 0));
    // the row's sum is the two halves' sums
    exch[row * 2 + half] = l;
    pair_sync();
    if (ok) {
      tc_fence_after();
      const float lt = exch[row * 2] + exch[row * 2 + 1];
      const float inv = lt > 0.0f ? 1.0f / lt : 0.0f;
#pragma unroll 1
      for (int c4 = 0; c4 < 2; ++c4) {
        float v[32];
        tmem_ld32(v, o_addr + 32 * c4);
        if (qpos < T) {
          float4* dst = reinterpret_cast<float4*>(out + ((static_cast<long long>(b) * T + qpos) * Hq + hq) * kHeadDim + 64 * half + 32 * c4);
#pragma unroll
          for (int e = 0; e < 32; e += 4) dst[e >> 2] = make_float4(v[e] * inv, v[e + 1] * inv, v[e + 2] * inv, v[e + 3] * inv);
        }
      }
    } else if (lane == 0) {
      set_status(cv.status, MOQAE_ERR_TIMEOUT, blockIdx.x, warp);
    }
  } else if (warp < kSoftmaxWarps) {
    // ================= softmax: one query row per thread =================
    const int i = warp >> 2;                        // query tile of this warp
    const int nb = i ? nb1 : nb0;
    const int row = tid & 127;
    const int qpos = (2 * pair + i) * kQTile + row;
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t s_addr = lane_addr + 128 * i, o_addr = lane_addr + 256 + 128 * i;
    // The reference maximum m_ref is an integer (base-2 units), so that a move of it rescales
    // what is already stored by an exact power of two.
    float m_ref = -INFINITY, l = 0.0f;
    bool ok = true;
    for (int kb = 0; kb < nb && ok; ++kb) {
      ok = __all_sync(0xffffffffu, wait(BAR_SFULL + i, kb));
      if (!ok) break;
      tc_fence_after();
      // Blocks left of the diagonal are fully visible; only the last one needs the mask.
      const bool diag = kb >= 2 * pair + i;
      const int rel = qpos - kb * kKvBlock;          // columns 0..rel of this block are visible
      float sum = 0.0f;
#pragma unroll 1
      for (int c4 = 0; c4 < kKvBlock / 32; ++c4) {
        float v[32];
        tmem_ld32(v, s_addr + 32 * c4);
        if (diag) {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (32 * c4 + e > rel) v[e] = -INFINITY;
        }
        // Weights against the current reference, with no look at the scores' maximum first: as
        // long as the chunk's sum stays below kSumLimit no weight can overflow fp16, and the
        // reference may lag the true maximum.
        uint32_t pk[16];
        float csum;
        auto weights = [&]() {
          const uint64_t scale2 = pack_f2(scale_log2, scale_log2), negm2 = pack_f2(-m_ref, -m_ref);
          uint64_t part[2] = {0ull, 0ull};           // two packed partial sums (even / odd columns each)
#pragma unroll
          for (int e2 = 0; e2 < 16; ++e2) {
            float x0, x1;
            unpack_f2(fma_f2(pack_f2(v[2 * e2], v[2 * e2 + 1]), scale2, negm2), x0, x1);
            const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
            part[e2 & 1] = add_f2(part[e2 & 1], pack_f2(p0, p1));
            pk[e2] = pack_h2(p0, p1);
          }
          float s0, s1;
          unpack_f2(add_f2(part[0], part[1]), s0, s1);
          csum = s0 + s1;
        };
        weights();
        if (__any_sync(0xffffffffu, !(csum < kSumLimit))) {
          // Rare (always on the very first chunk, where the reference is still -inf): some row of
          // the warp met scores far above its reference.  Move the reference to the chunk's maximum
          // and rescale what was accumulated against the old one: O_i (at rest: S_i of this block
          // was issued after the last O_i += P_i V^), the running sums, and the chunks of P_i already
          // written for this block; then form this chunk's weights again.
          float mx = v[0];
#pragma unroll
          for (int e = 1; e < 32; ++e) mx = fmaxf(mx, v[e]);
          mx *= scale_log2;                          // scale_log2 > 0
          const float m_new = fmaxf(m_ref, ceilf(mx));
          const float corr = (m_ref == -INFINITY) ? 0.0f : ex2_approx(m_ref - m_new);
          if (kb > 0) {
#pragma unroll 1
            for (int o4 = 0; o4 < 4; ++o4) {
              float o[32];
              tmem_ld32(o, o_addr + 32 * o4);
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] *= corr;
              tmem_st32(o_addr + 32 * o4, o);
            }
          }
          tmem_st_wait();
#pragma unroll 1
          for (int p4 = 0; p4 < c4; ++p4) {
            uint32_t pw[16];
            tmem_ld16u(pw, s_addr + 16 * p4);
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&pw[e]));
              pw[e] = pack_h2(f.x * corr, f.y * corr);
            }
            tmem_st16u_nowait(s_addr + 16 * p4, pw);
          }
          l *= corr;
          sum *= corr;
          m_ref = m_new;
          weights();
        }
        sum += csum;
        tmem_st16u_nowait(s_addr + 16 * c4, pk);     // columns already read: 16 (c4 + 1) <= 32 (c4 + 1)
      }
      l += sum;
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BAR_PFULL + i));
    }
    if (ok && nb > 0) ok = __all_sync(0xffffffffu, wait(BAR_OFULL + i, 0));
    if (ok) {
      tc_fence_after();
      const float inv = l > 0.0f ? 1.0f / l : 0.0f;
#pragma unroll 1
      for (int c4 = 0; c4 < 4; ++c4) {
        float v[32];
        tmem_ld32(v, o_addr + 32 * c4);
        if (qpos < T) {
          float4* dst = reinterpret_cast<float4*>(out + ((static_cast<long long>(b) * T + qpos) * Hq + hq) * kHeadDim + 32 * c4);
#pragma unroll
          for (int e = 0; e < 32; e += 4) dst[e >> 2] = make_float4(v[e] * inv, v[e + 1] * inv, v[e + 2] * inv, v[e + 3] * inv);
        }
      }
    } else if (lane == 0) {
      set_status(cv.status, MOQAE_ERR_TIMEOUT, blockIdx.x, warp);
    }
  } else if (PRE && warp > kIssueWarp) {
    // ================= fetch: K^ (warp 17) and V^ (warp 18) blocks from the fp16 scratch by TMA =================
    if (lane == 0) {
      const bool is_v = warp == kIssueWarp + 2;
      const CUtensorMap* map = is_v ? &map_v : &map_k;
      const int row0 = (b * H + h) * t_pad;
      for (int kb = 0; kb < nb1; ++kb) {
        const int st = kb % kStages;
        if (kb >= kStages && !wait((is_v ? BAR_VFREE : BAR_KFREE) + st, kb / kStages - 1)) break;
        const uint32_t full = bar((is_v ? BAR_VFULL : BAR_KFULL) + st);
        const uint32_t dst = smem_u32((is_v ? sV : sK) + st * kStageBytes);
        mbar_expect_tx(full, kStageBytes);
        tma_load_2d(dst, map, 0, row0 + kb * kKvBlock, full);                    // channels 0..63
        tma_load_2d(dst + kStageBytes / 2, map, 64, row0 + kb * kKvBlock, full);  // channels 64..127
      }
    }
  } else if (warp < kIssueWarp) {
    // ================= dequantise: storage tile `sub` of every block =================
    const int dw = warp - kSoftmaxWarps;
    const bool is_v = dw >= 4;
    const int sub = dw & 3;
    const KvSource ks = kv_source(cv, dm, layer, b, h);
    for (int kb = 0; kb < nb1; ++kb) {
      const int st = kb % kStages;
      const int pos0 = kb * kKvBlock + sub * kTileTokens;
      // the stage is free once the products that read it kStages blocks back are done
      if (kb >= kStages && !wait((is_v ? BAR_VFREE : BAR_KFREE) + st, kb / kStages - 1)) break;
      dequant_subtile<BF16, false>(ks, pos0, sub, is_v, (is_v ? sV : sK) + st * kStageBytes, lane);
      fence_async_proxy();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar((is_v ? BAR_VFULL : BAR_KFULL) + st));
    }
  } else {
    // ================= MMA issue (one thread) =================
    // descriptors of stage 0, K step 0; a stage adds kStageBytes / 16 to the low word, a K step
    // (two 2 KiB slabs of 8 channels or 8 tokens) 256
    const uint64_t qd = make_desc(smem_u32(sQ), 2048, 128);
    const uint64_t kd = PRE ? make_desc_sw128(smem_u32(sK), 16, 1024) : make_desc(smem_u32(sK), 2048, 128);
    const uint64_t vd = PRE ? make_desc_sw128(smem_u32(sV), kStageBytes / 2, 1024) : make_desc(smem_u32(sV), 2048, 128);
    const uint32_t qd_lo = static_cast<uint32_t>(qd), qd_hi = static_cast<uint32_t>(qd >> 32);
    const uint32_t kd_lo = static_cast<uint32_t>(kd), kd_hi = static_cast<uint32_t>(kd >> 32);
    const uint32_t vd_lo = static_cast<uint32_t>(vd), vd_hi = static_cast<uint32_t>(vd >> 32);
    // S_i = Q_i K^[st]^T: K = 128 channels in 8 steps of 16; the last product that reads K^[st]
    // (tile 1) also frees the stage
    auto issue_s = [&](int i, int kb) {
      const int st = kb % kStages;
      if (lane == 0) {
        const uint32_t a_lo = qd_lo + i * (kQTileBytes >> 4), b_lo = kd_lo + st * (kStageBytes >> 4), d = tmem + 128 * i;
#pragma unroll
        for (int k = 0; k < 8; ++k)   // K step of the swizzled K^: 32 bytes inside the row, 16 KiB to the second half of the channels
          umma_f16_ss(d, a_lo + 256 * k, qd_hi, b_lo + (PRE ? (k >> 2) * 1024 + (k & 3) * 2 : 256 * k), kd_hi, kIdescS, k > 0);
        umma_commit(bar(BAR_SFULL + i));
        if (i == 1) umma_commit(bar(BAR_KFREE + st));
      }
      __syncwarp();
    };
    // O_i += P_i V^[st]: K = 128 tokens in 8 steps of 16
    auto issue_pv = [&](int i, int kb, bool last) {
      const int st = kb % kStages;
      if (lane == 0) {
        const uint32_t lo = vd_lo + st * (kStageBytes >> 4), d = tmem + 256 + 128 * i, a = tmem + 128 * i;
        umma_f16_ta(d, a, lo, vd_hi, kIdescPV, kb > 0);
#pragma unroll
        for (int k = 1; k < 8; ++k)   // K step of the swizzled V^: 16 token rows of 128 bytes
          umma_f16_ta(d, a + 8 * k, lo + (PRE ? 128 : 256) * k, vd_hi, kIdescPV, 1u);
        if (i == 1) umma_commit(bar(BAR_VFREE + st));
        if (last) umma_commit(bar(BAR_OFULL + i));
      }
      __syncwarp();
    };
    bool ok = wait(BAR_KFULL, 0);
    if (ok) {
      tc_fence_after();
      issue_s(0, 0);
      issue_s(1, 0);
    }
    // Block kb, tile by tile: O_i += P_i V^ as soon as P_i is there, then at once S_i of the next
    // block; the other tile's products run while this tile's softmax threads work on it.
    for (int kb = 0; kb < nb1 && ok; ++kb) {
      ok = wait(BAR_VFULL + kb % kStages, kb / kStages);
      if (ok && kb + 1 < nb1) ok = wait(BAR_KFULL + (kb + 1) % kStages, (kb + 1) / kStages);
      for (int i = 0; i < 2 && ok; ++i) {
        const int nb = i ? nb1 : nb0;
        if (kb >= nb) continue;
        ok = wait(BAR_PFULL + i, kb);
        if (!ok) break;
        tc_fence_after();
        issue_pv(i, kb, kb + 1 == nb);
        if (kb + 1 < nb) issue_s(i, kb + 1);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kIssueWarp)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols2) : "memory");
}

}  // namespace

// [rows][128] fp16 rows, boxes of 64 channels x 128 rows, 128-byte swizzle
static bool make_block_map(CUtensorMap* m, const void* base, long long rows) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t gdim[2] = {kHeadDim, static_cast<cuuint64_t>(rows)};
  const cuuint64_t gstride[1] = {kHeadDim * 2};
  const cuuint32_t box[2] = {64, kKvBlock};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int padded_tokens(int T) { return (T + kKvBlock - 1) / kKvBlock * kKvBlock; }

long long prefill_workspace_bytes(const Dims& dm, int T) {
  return 2ll * dm.batch * dm.n_kv_heads * padded_tokens(T) * kHeadDim * 2;
}

template <bool BF16, bool PRE>
static cudaError_t launch_attn(const Dims& dm, const CacheView& cv, const void* q, int T, int layer, float scale, float* out,
                               const CUtensorMap& mk, const CUtensorMap& mv, int t_pad, cudaStream_t st) {
  const size_t smem = 1024 + 2 * kQTileBytes + 2 * kStages * kStageBytes + BAR_COUNT * 8 + 16 + kExchangeBytes;
  dim3 grid((T + 2 * kQTile - 1) / (2 * kQTile), dm.n_q_heads, dm.batch);
  cudaError_t e = cudaFuncSetAttribute(prefill_attn_kernel<BF16, PRE>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  prefill_attn_kernel<BF16, PRE><<<grid, block_threads(PRE), smem, st>>>(dm, cv, static_cast<const uint16_t*>(q), T, layer,
                                                                 scale * 1.4426950408889634f, out, mk, mv, t_pad);
  return cudaGetLastError();
}

// workspace == nullptr: every CTA expands the packed tiles itself (no extra memory).  Otherwise the
// layer is expanded once into the workspace (prefill_workspace_bytes) and fetched from there.
cudaError_t launch_prefill_attn(const Dims& dm, const CacheView& cv, const void* q, int T, int layer, float scale,
                                float* out, void* workspace, cudaStream_t st) {
  if (T <= 0) return cudaSuccess;
  const bool bf16 = dm.dtype == MOQAE_DTYPE_BF16;
  CUtensorMap mk, mv;
  memset(&mk, 0, sizeof(mk));
  memset(&mv, 0, sizeof(mv));
  if (!workspace)
    return bf16 ? launch_attn<true, false>(dm, cv, q, T, layer, scale, out, mk, mv, 0, st)
                : launch_attn<false, false>(dm, cv, q, T, layer, scale, out, mk, mv, 0, st);
  const int t_pad = padded_tokens(T);
  uint8_t* kd = static_cast<uint8_t*>(workspace);
  uint8_t* vd = kd + prefill_workspace_bytes(dm, T) / 2;
  const long long rows = static_cast<long long>(dm.batch) * dm.n_kv_heads * t_pad;
  if (!make_block_map(&mk, kd, rows) || !make_block_map(&mv, vd, rows)) return cudaErrorNotSupported;
  dim3 dgrid(t_pad / kTileTokens, dm.n_kv_heads, dm.batch);
  if (bf16) prefill_dequant_kernel<true><<<dgrid, 64, 0, st>>>(dm, cv, layer, t_pad, kd, vd);
  else prefill_dequant_kernel<false><<<dgrid, 64, 0, st>>>(dm, cv, layer, t_pad, kd, vd);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return bf16 ? launch_attn<true, true>(dm, cv, q, T, layer, scale, out, mk, mv, t_pad, st)
              : launch_attn<false, true>(dm, cv, q, T, layer, scale, out, mk, mv, t_pad, st);
}

}  // namespace moqae
