// Split-K decode attention, tensor-core version (the production path).
//
// Each warp is an independent stream processor: it owns a private ring of shared-memory
// stages that one elected lane fills with 1-D bulk copies (cp.async.bulk + mbarrier
// complete_tx), and it consumes whole tiles from that ring.  Per 32-token tile:
//
//   scores   S[t][q] = sum_c code[t][c] * (q[c] s_k[c]) + sum_c q[c] z_k[c]
//            The codes are never converted: a payload word (or the word shifted right by 8)
//            masked at one code position in both half-words IS a pair of fp16 subnormals
//            (code * 2^pos * 2^-24), the power of two and the key scale are folded into the
//            query fragment once per tile, and the product runs on mma.sync m16n8k16
//            (A = 16 tokens x 16 channels of codes, B = folded queries of the GQA group
//            padded to 8 columns, fp32 accumulate).  The zero-point term is a second MMA
//            chain with exact fp16 operands (A = z_k, B = q).
//   softmax  online, base 2, in registers, with a lazily moved reference maximum; weights are
//            kept <= 64 so that p*s_v stays in fp16 range.
//   output   out[c][q] = sum_t code[t][c] * (p[t][q] s_v[t][cg]) + sum_t p[t][q] z_v[t][cg]
//            again with untouched codes as the A operand (A = V^T, 16 channels x 16 tokens:
//            the value payload stores, per lane, words of 4 tokens of each channel row it
//            owns), P transposed in registers with movmatrix, one extra MMA for the zero
//            term.  Code positions differ only between accumulator rows, so they are undone
//            once per phase on the accumulators.
//   The storage format puts every 16-byte unit where the lane that needs it reads it:
//   all shared-memory reads of a tile are conflict-free 128-bit loads.
//
// 16-bit tiles and the 16-bit tail run the same MMAs on the raw values.
// Every wait on an mbarrier is bounded; on expiry the warp records MOQAE_ERR_TIMEOUT in
// the cache's status word and stops consuming.
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace moqae {

namespace {

constexpr int kWarps = 6;
constexpr int kThreads = kWarps * 32;
constexpr int kRingBytes = 18432;             // per warp: 6 x 3 KiB = 3 x 5 KiB(+) = 2 x 9 KiB = 2 x 8 KiB(+)
constexpr int kQBytes = 8 * kHeadDim * 2;     // one 8-query fragment source, 16-bit
template <bool BF16>
__device__ __forceinline__ void mma16816(float d[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  if (BF16) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t r;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(r) : "r"(x));
  return r;
}
__device__ __forceinline__ float ex2f(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ uint32_t hmul2_u32(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("mul.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
// a*b - c in one rounding: with c = round(a*b) this is the exact rounding error of the product
__device__ __forceinline__ uint32_t hfma2_sub_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("{\n.reg .b32 n;\nneg.f16x2 n, %3;\nfma.rn.f16x2 %0, %1, %2, n;\n}\n" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_bf162(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// ---- code extraction: masked words are pairs of fp16 subnormals ------------------------
// A 32-bit payload word holds n = 32/BITS codes, code i at bits [BITS*i, BITS*i + BITS).
// Register (s, m) of a word is ((s ? w >> 8 : w) & (mask << BITS*m)): its low half-word is
// code s*(n/4) + m, its high half-word code s*(n/4) + m + n/2, both at bit position BITS*m.
template <int BITS> struct Fmt {
  static constexpr int n = 32 / BITS;                 // codes per word
  static constexpr int regs = n / 2;                  // registers per word
  static constexpr int direct = n / 4;                // of which taken from the unshifted word
  static constexpr uint32_t mask = ((1u << BITS) - 1u) * 0x00010001u;
};
template <int BITS> __device__ __forceinline__ uint32_t ext(uint32_t w, uint32_t wsh, int s, int m) {
  return (s ? wsh : w) & (Fmt<BITS>::mask << (BITS * m));
}
// register number r (0..15) of a 32-channel key piece -> word j, shifted?, position m
template <int BITS> __host__ __device__ constexpr int reg_word(int r) { return r / Fmt<BITS>::regs; }
template <int BITS> __host__ __device__ constexpr int reg_shifted(int r) { return (r % Fmt<BITS>::regs) / Fmt<BITS>::direct; }
template <int BITS> __host__ __device__ constexpr int reg_m(int r) { return r % Fmt<BITS>::direct; }
// channel (inside the piece) of the low half of register r; the high half is n/2 further
template <int BITS> __host__ __device__ constexpr int reg_channel_lo(int r) {
  return reg_word<BITS>(r) * Fmt<BITS>::n + reg_shifted<BITS>(r) * Fmt<BITS>::direct + reg_m<BITS>(r);
}
// fp16 constant 2^e as a half2 bit pattern (e in the normal range)
__host__ __device__ constexpr uint32_t half2_pow2(int e) {
  return (static_cast<uint32_t>(e + 15) << 10) | (static_cast<uint32_t>(e + 15) << 26);
}

struct State {
  float acc[8][4];   // M-tile mt = 2*cg + hf: rows g / g+8 = channels 32cg+4g+2hf / +1; cols = queries 2t4, 2t4+1
  float oz[4];       // rows 0..3 (lanes g < 4): zero-point term per channel group; row 4 (g == 4): the
                     // running sums l, taken over the SAME rounded weights the values are multiplied by
  float m[2];        // reference maxima (base-2 exponent units) of queries 2t4, 2t4+1
};

// Per-lane constants of the quantised phases.  Every query row is normalised by a power of two,
// q' = q * 2^-e with |q'| < 1, before it becomes an fp16 operand, so that q' * s_k can never leave
// the fp16 range whatever the key scale is; the power of two comes back, exactly, in these factors.
struct LaneConst {
  float cs[2];       // raw score sum (units of 2^-24 * 2^-e) -> base-2 logits, queries 2t4 and 2t4+1
  float cbg;         // the same for the zero-point term of query g (no 2^-24 there)
};

__device__ __forceinline__ void rescale(State& st, float c0, float c1) {
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    st.acc[mt][0] *= c0; st.acc[mt][1] *= c1; st.acc[mt][2] *= c0; st.acc[mt][3] *= c1;
  }
  st.oz[0] *= c0; st.oz[1] *= c1; st.oz[2] *= c0; st.oz[3] *= c1;
}

// Online softmax with a lazily moved reference maximum m: only when some score exceeds m by more
// than kSlack does the warp reduce the true maximum (three shuffle rounds) and rescale its
// accumulators; otherwise m stays.  Weights are p~ = 2^(x - m + PK - kSlack) <= 2^PK, with PK
// chosen per width so that p~ * s_v cannot leave the fp16 range for any scale the quantiser can
// produce (s_v <= 65504 / (2^b - 1)) while typical products stay well above the subnormals:
// 2^1 * 21835, 2^3 * 4367, 2^7 * 257 < 65504.  Between phases the state is kept at PK = 0.
constexpr float kSlack = 3.0f;
template <int BITS> __host__ __device__ constexpr int pmax_log2() { return BITS == 2 ? 1 : BITS == 4 ? 3 : BITS == 8 ? 7 : 6; }

// The same for a query group of at most 4, where a lane's even column (2 t4) is query t4 and its odd column is
// not used: xm0 = this lane's largest score of that query.
__device__ __forceinline__ void move_reference_even(State& st, float xm0) {
  if (__any_sync(0xffffffffu, xm0 > st.m[0] + kSlack)) {
#pragma unroll
    for (int o = 4; o <= 16; o <<= 1) xm0 = fmaxf(xm0, __shfl_xor_sync(0xffffffffu, xm0, o));
    const float n0 = fmaxf(st.m[0], xm0);
    const float c0 = (st.m[0] == -INFINITY) ? 0.0f : ex2f(st.m[0] - n0);
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      st.acc[mt][0] *= c0; st.acc[mt][1] *= c0; st.acc[mt][2] *= c0; st.acc[mt][3] *= c0;
    }
    st.oz[0] *= c0; st.oz[1] *= c0; st.oz[2] *= c0; st.oz[3] *= c0;
    st.m[0] = n0;
  }
}

// xm0 / xm1: this lane's largest scores of queries 2t4 / 2t4+1 in the unit about to be weighted
__device__ __forceinline__ void move_reference(State& st, float xm0, float xm1) {
  const bool over = (xm0 > st.m[0] + kSlack) || (xm1 > st.m[1] + kSlack);
  if (__any_sync(0xffffffffu, over)) {
#pragma unroll
    for (int o = 4; o <= 16; o <<= 1) {
      xm0 = fmaxf(xm0, __shfl_xor_sync(0xffffffffu, xm0, o));
      xm1 = fmaxf(xm1, __shfl_xor_sync(0xffffffffu, xm1, o));
    }
    const float n0 = fmaxf(st.m[0], xm0), n1 = fmaxf(st.m[1], xm1);
    const float c0 = (st.m[0] == -INFINITY) ? 0.0f : ex2f(st.m[0] - n0);
    const float c1 = (st.m[1] == -INFINITY) ? 0.0f : ex2f(st.m[1] - n1);
    rescale(st, c0, c1);
    st.m[0] = n0; st.m[1] = n1;
  }
}

// Update for NV score vectors x[v][4] (d-fragment order: row g q0, row g q1, row g+8 q0,
// row g+8 q1; already in base-2 units; -inf = masked).  Returns the weights p~ in x.
template <int NV>
__device__ __forceinline__ void softmax_update(State& st, float x[NV][4]) {
  constexpr float kPmaxLog2 = static_cast<float>(pmax_log2<16>());
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    mx0 = fmaxf(mx0, fmaxf(x[v][0], x[v][2]));
    mx1 = fmaxf(mx1, fmaxf(x[v][1], x[v][3]));
  }
  move_reference(st, mx0, mx1);
  const float o0 = (kPmaxLog2 - kSlack) - st.m[0], o1 = (kPmaxLog2 - kSlack) - st.m[1];
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    x[v][0] = ex2f(x[v][0] + o0); x[v][1] = ex2f(x[v][1] + o1);
    x[v][2] = ex2f(x[v][2] + o0); x[v][3] = ex2f(x[v][3] + o1);
  }
}

// ---- NT quantised tiles (32 tokens each) from shared memory ----------------------------
// Lane (g, t4) = (lane / 4, lane % 4).  qb[r], r = 0..15: fp16 pair (q'[c_lo(r)], q'[c_hi(r)])
// of query g (zero for g >= G) for the channels 32*t4 + .. that key register r carries;
// qc[r] = qb[r] times the power of two that undoes the register's bit position.
// G4 (query group of at most 4): B column 2q carries the high part and column 2q + 1 the low part of
// folded query q, so one MMA chain yields both halves of the exact product and lane (g, t4) finds
// the two halves of query t4 side by side in its own accumulator registers.  Everything after the
// scores then works on the lane's even column only (one query per lane, half the weights to
// compute); for quantised tiles the odd columns of P are zero, 16-bit bf16 tiles put the low parts of their
// weights there, and a query's result is its even plus its odd accumulator column.
// NT = 2 (neighbouring 2-bit tiles, fetched by one copy): one reference-maximum check, one set of
// zero-point MMAs and one round of bias shuffles serve both tiles.
template <int BITS, int NT, bool G4>
__device__ __forceinline__ void process_qunit(const uint8_t* __restrict__ unit, State& st,
                                              const uint32_t (&qc)[16], const uint32_t (&qb)[16],
                                              const LaneConst& lc, int lane, int n_valid) {
  using F = Fmt<BITS>;
  constexpr int TB = kMetaBytes + 1024 * BITS;       // bytes per tile
  constexpr int NB = 2 * NT;                         // 16-token blocks
  const int g = lane >> 2, t4 = lane & 3;

  // fold the key scales into the query fragments: q'*s = hi + lo exactly (two fp16 each), so the
  // scores carry no rounding besides the fp32 accumulation
  uint32_t qf[NT][16], ql[G4 ? 1 : NT][G4 ? 1 : 16];
#pragma unroll
  for (int tl = 0; tl < NT; ++tl) {
    const uint4* sp = reinterpret_cast<const uint4*>(unit + tl * TB) + t4;
    const bool lo_lane = G4 && (g & 1);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint4 s4 = sp[4 * i];
      const uint32_t sv[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t hi = hmul2_u32(qc[4 * i + j], sv[j]);
        if (G4) {
          // lanes of the odd columns replace hi by lo = fma(q', s, -hi)
          if (lo_lane) hi = hfma2_sub_u32(qc[4 * i + j], sv[j], hi);
        } else {
          ql[G4 ? 0 : tl][(4 * i + j) % (G4 ? 1 : 16)] = hfma2_sub_u32(qc[4 * i + j], sv[j], hi);
        }
        qf[tl][4 * i + j] = hi;
      }
    }
  }

  // key payload words of every 16-token block: w[b2][hh][j], hh = rows g / g + 8
  uint32_t w[NB][2][BITS];
#pragma unroll
  for (int b2 = 0; b2 < NB; ++b2) {
    const uint8_t* kpay = unit + (b2 >> 1) * TB + kMetaBytes;
    const int blk = b2 & 1;
    if (BITS == 2) {
      const uint4 u = *reinterpret_cast<const uint4*>(kpay + (blk * 32 + lane) * 16);
      w[b2][0][0] = u.x; w[b2][0][1] = u.y; w[b2][1][0] = u.z; w[b2][1][1] = u.w;
    } else if (BITS == 4) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const uint4 u = *reinterpret_cast<const uint4*>(kpay + ((2 * blk + hh) * 32 + lane) * 16);
        w[b2][hh][0] = u.x; w[b2][hh][1] = u.y; w[b2][hh][2 % BITS] = u.z; w[b2][hh][3 % BITS] = u.w;
      }
    } else {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int j2 = 0; j2 < 2; ++j2) {
          const uint4 u = *reinterpret_cast<const uint4*>(kpay + (((2 * blk + hh) * 2 + j2) * 32 + lane) * 16);
          w[b2][hh][(4 * j2) % BITS] = u.x; w[b2][hh][(4 * j2 + 1) % BITS] = u.y;
          w[b2][hh][(4 * j2 + 2) % BITS] = u.z; w[b2][hh][(4 * j2 + 3) % BITS] = u.w;
        }
    }
  }

  // Zero-point term of the scores: bias[tile][q] = sum_c z_k[c] q'[c], exact products.  The
  // queries are the A operand (rows g and g + 8 both hold query g: registers 4i, 4i+2 in row g,
  // 4i+1, 4i+3 in row g + 8), the zeros the B operand.  B column n carries, for tile (n & 3) >> 1
  // (NT = 2) or the only tile, the zeros of registers 4i, 4i+2 (n even) or 4i+1, 4i+3 (n odd);
  // the zero array stores each group of four registers in the order 0, 2, 1, 3.  Element
  // (g, n even) + element (g + 8, n + 1) is then the full sum for query g: lane (g, t4) finds
  // both in its own fragment, for tile t4 & 1 (NT = 2).
  float bd[4] = {0.f, 0.f, 0.f, 0.f};
  const uint8_t* zp = unit + (NT == 2 ? ((g & 3) >> 1) * TB : 0) + 256 + t4 * 16 + (g & 1) * 8;

  // Raw score sums of the NB blocks (rows g and g + 8 of each).  Step i of a block multiplies key
  // registers 2i, 2i+1 (made from the payload words right before use) with the folded query; the
  // steps of all blocks are interleaved so that four independent accumulator chains are always in
  // flight, and the four zero-point MMAs ride along.
  constexpr int CH = 4 / NB;                         // accumulator chains per block
  float sc[NB][CH][4];
#pragma unroll
  for (int b2 = 0; b2 < NB; ++b2)
#pragma unroll
    for (int c = 0; c < CH; ++c)
#pragma unroll
      for (int i = 0; i < 4; ++i) sc[b2][c][i] = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
#pragma unroll
    for (int b2 = 0; b2 < NB; ++b2) {
      uint32_t a[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int r = 2 * i + (k >> 1), hh = k & 1;            // a0: (r0, hh0) a1: (r0, hh1) a2: (r1, hh0) a3: (r1, hh1)
        const int j = r / F::regs, rr = r % F::regs;
        const uint32_t word = w[b2][hh][j];
        a[k] = ext<BITS>(word, word >> 8, rr / F::direct, rr % F::direct);
      }
      const int tl = b2 >> 1;
      mma16816<false>(sc[b2][i % CH], a[0], a[1], a[2], a[3], qf[tl][2 * i], qf[tl][2 * i + 1]);
      if (!G4) {
        constexpr int M = G4 ? 1 : 16;
        mma16816<false>(sc[b2][i % CH], a[0], a[1], a[2], a[3], ql[G4 ? 0 : tl][(2 * i) % M], ql[G4 ? 0 : tl][(2 * i + 1) % M]);
      }
    }
    if (i & 1) {
      const int k = i >> 1;
      const uint2 z = *reinterpret_cast<const uint2*>(zp + 64 * k);
      mma16816<false>(bd, qb[4 * k], qb[4 * k + 1], qb[4 * k + 2], qb[4 * k + 3], z.x, z.y);
    }
  }
  float bias[NT][2];
  {
    const float bq = (bd[0] + bd[3]) * lc.cbg;            // query of row g, tile t4 & 1
#pragma unroll
    for (int tl = 0; tl < NT; ++tl) {
      bias[tl][0] = __shfl_sync(0xffffffffu, bq, 8 * t4 + (NT == 2 ? tl : 0));
      bias[tl][1] = G4 ? 0.0f : __shfl_sync(0xffffffffu, bq, 8 * t4 + 4 + (NT == 2 ? tl : 0));
    }
  }
  float v[NB][4];
#pragma unroll
  for (int b2 = 0; b2 < NB; ++b2)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float x = sc[b2][0][i];
      if (CH == 2) x += sc[b2][CH - 1][i];
      v[b2][i] = x;
    }
  if (G4) {
    // high part (even column) + low part (odd column) of the lane's query, rows g and g + 8
#pragma unroll
    for (int b2 = 0; b2 < NB; ++b2) {
      v[b2][0] += v[b2][1];
      v[b2][2] += v[b2][3];
    }
  }
  if (n_valid < kTileTokens) {
    // tiles of a chunk shorter than 32 tokens: positions n_valid (8 or 16) .. 31 are padding and get
    // weight zero (row g of block 0 is token g, row g + 8 token g + 8, block 1 tokens 16..31)
#pragma unroll
    for (int b2 = 0; b2 < NB; ++b2) {
      const bool lo_ok = (b2 & 1) == 0, hi_ok = (b2 & 1) == 0 && n_valid > 8;
      if (!lo_ok) v[b2][0] = v[b2][1] = -INFINITY;
      if (!hi_ok) v[b2][2] = v[b2][3] = -INFINITY;
    }
  }

  // softmax: the factor cs > 0 and the per-tile bias commute with the maximum, so the reference
  // check runs on the raw sums and every weight costs one FMA and one ex2
  if (G4) {
    float xm0 = -INFINITY;
#pragma unroll
    for (int tl = 0; tl < NT; ++tl) {
      const float r0 = fmaxf(fmaxf(v[2 * tl][0], v[2 * tl][2]), fmaxf(v[2 * tl + 1][0], v[2 * tl + 1][2]));
      xm0 = fmaxf(xm0, fmaf(r0, lc.cs[0], bias[tl][0]));
    }
    move_reference_even(st, xm0);
    constexpr float kPmaxLog2 = static_cast<float>(pmax_log2<BITS>());
    const float o0 = (kPmaxLog2 - kSlack) - st.m[0];
#pragma unroll
    for (int tl = 0; tl < NT; ++tl) {
      const float ob0 = bias[tl][0] + o0;
#pragma unroll
      for (int blk = 0; blk < 2; ++blk) {
        float* x = v[2 * tl + blk];
        x[0] = ex2f(fmaf(x[0], lc.cs[0], ob0)); x[1] = 0.0f;
        x[2] = ex2f(fmaf(x[2], lc.cs[0], ob0)); x[3] = 0.0f;
      }
    }
  } else {
    float xm0 = -INFINITY, xm1 = -INFINITY;
#pragma unroll
    for (int tl = 0; tl < NT; ++tl) {
      const float r0 = fmaxf(fmaxf(v[2 * tl][0], v[2 * tl][2]), fmaxf(v[2 * tl + 1][0], v[2 * tl + 1][2]));
      const float r1 = fmaxf(fmaxf(v[2 * tl][1], v[2 * tl][3]), fmaxf(v[2 * tl + 1][1], v[2 * tl + 1][3]));
      xm0 = fmaxf(xm0, fmaf(r0, lc.cs[0], bias[tl][0]));
      xm1 = fmaxf(xm1, fmaf(r1, lc.cs[1], bias[tl][1]));
    }
    move_reference(st, xm0, xm1);
    constexpr float kPmaxLog2 = static_cast<float>(pmax_log2<BITS>());
    const float o0 = (kPmaxLog2 - kSlack) - st.m[0], o1 = (kPmaxLog2 - kSlack) - st.m[1];
#pragma unroll
    for (int tl = 0; tl < NT; ++tl) {
      const float ob0 = bias[tl][0] + o0, ob1 = bias[tl][1] + o1;
#pragma unroll
      for (int blk = 0; blk < 2; ++blk) {
        float* x = v[2 * tl + blk];
        x[0] = ex2f(fmaf(x[0], lc.cs[0], ob0)); x[1] = ex2f(fmaf(x[1], lc.cs[1], ob1));
        x[2] = ex2f(fmaf(x[2], lc.cs[0], ob0)); x[3] = ex2f(fmaf(x[3], lc.cs[1], ob1));
      }
    }
  }

#pragma unroll
  for (int b2 = 0; b2 < NB; ++b2) {
    const uint8_t* tile = unit + (b2 >> 1) * TB;
    const uint8_t* vpay = tile + kMetaBytes + kTileTokens * 16 * BITS;
    const int blk = b2 & 1;
    const uint32_t p0 = movmatrix_trans(pack_half2(v[b2][0], v[b2][1]));   // tokens 16blk + 2t4, +1 of query g
    const uint32_t p1 = movmatrix_trans(pack_half2(v[b2][2], v[b2][3]));   // tokens 16blk + 8 + 2t4, +1
    {  // zero-point term: rows = channel groups (lanes g < 4)
      uint32_t z0 = (g == 4) ? 0x3C003C00u : 0u, z1 = z0;      // row 4: ones -> sum of the weights
      if (g < 4) {
        const uint2 z = *reinterpret_cast<const uint2*>(tile + 768 + ((blk * 4 + g) * 4 + t4) * 8);
        z0 = z.x; z1 = z.y;
      }
      mma16816<false>(st.oz, z0, 0u, z1, 0u, p0, p1);
    }
    uint32_t pb[4][2];
#pragma unroll
    for (int cp = 0; cp < 2; ++cp) {
      const uint4 sv = *reinterpret_cast<const uint4*>(tile + 512 + ((blk * 2 + cp) * 4 + t4) * 16);
      pb[2 * cp][0] = hmul2_u32(p0, sv.x); pb[2 * cp][1] = hmul2_u32(p1, sv.y);
      pb[2 * cp + 1][0] = hmul2_u32(p0, sv.z); pb[2 * cp + 1][1] = hmul2_u32(p1, sv.w);
    }
    // value words of this lane: channel rows R = 0..15 (channel 32*(R/4) + 4g + R%4), 4 tokens each
    constexpr int NW = 2 * BITS;
    uint32_t wv[NW];
#pragma unroll
    for (int u = 0; u < BITS / 2; ++u) {
      const uint4 x4 = *reinterpret_cast<const uint4*>(vpay + ((blk * (BITS / 2) + u) * 32 + lane) * 16);
      wv[4 * u] = x4.x; wv[4 * u + 1] = x4.y; wv[4 * u + 2] = x4.z; wv[4 * u + 3] = x4.w;
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      // rows R = 2mt (accumulator row g) and 2mt + 1 (row g + 8)
      constexpr int per = 8 / BITS;                      // rows per word
      const int w0 = (2 * mt) / per, sl0 = (2 * mt) % per;
      const int w1 = (2 * mt + 1) / per, sl1 = (2 * mt + 1) % per;
      const uint32_t m0 = F::mask << (BITS * sl0), m1 = F::mask << (BITS * sl1);
      mma16816<false>(st.acc[mt], wv[w0] & m0, wv[w1] & m1, (wv[w0] >> 8) & m0, (wv[w1] >> 8) & m1,
                      pb[mt >> 1][0], pb[mt >> 1][1]);
    }
  }
}

// power of two that accumulator row `hi` (0: row g, 1: row g + 8) of M-tile mt carries inside
// a quantised phase, in units of one code (the codes themselves are 2^-24 subnormals)
template <int BITS> __host__ __device__ constexpr int v_bitpos(int mt, int hi) {
  return BITS >= 16 ? 0 : BITS * ((2 * mt + hi) % (BITS >= 16 ? 1 : 8 / BITS));
}
// Entering a phase brings the state from the neutral units into the phase's (weights scaled by
// 2^PK everywhere, and for quantised widths the accumulator rows by their code position); leaving
// undoes it.  All factors are powers of two.
template <int BITS>
__device__ __forceinline__ void phase_scale(State& st, bool enter) {
  constexpr int pk = pmax_log2<BITS>();
#pragma unroll
  for (int mt = 0; mt < 8; ++mt)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = (BITS == 16 ? 0 : v_bitpos<BITS>(mt, i >> 1) - 24) + pk;     // accumulator = true * 2^e
      st.acc[mt][i] *= enter ? exp2f(static_cast<float>(e)) : exp2f(static_cast<float>(-e));
    }
#pragma unroll
  for (int i = 0; i < 4; ++i) st.oz[i] *= enter ? exp2f(static_cast<float>(pk)) : exp2f(static_cast<float>(-pk));
}

// Query fragments of a quantised phase: qb[r] = (q[c_lo(r)], q[c_hi(r)]) of query g as fp16,
// qc[r] = qb[r] * 2^(-bit position of register r).
template <int BITS>
__device__ __forceinline__ void load_q_phase(uint32_t (&qb)[16], uint32_t (&qc)[16], const uint16_t* q_h, int g, int t4) {
  const uint16_t* qrow = q_h + g * kHeadDim + 32 * t4;
#pragma unroll
  for (int r = 0; r < 16; ++r) {
    const int lo = reg_channel_lo<BITS>(r);
    qb[r] = static_cast<uint32_t>(qrow[lo]) | (static_cast<uint32_t>(qrow[lo + Fmt<BITS>::n / 2]) << 16);
    qc[r] = hmul2_u32(qb[r], half2_pow2(-BITS * reg_m<BITS>(r)));
  }
}

// ---- 16 raw rows (pool tile half or tail block) from shared memory ---------------------
// ks/vs: 16 rows x 256 B, 16-byte units swizzled by (row & 7).  qr[r]: q pairs of the raw
// channel set (units 2t4, 2t4+1, 8+2t4, 9+2t4) in the INPUT dtype.
template <bool BF16, bool G4>
__device__ __forceinline__ void process_raw16(const uint8_t* __restrict__ ks, const uint8_t* __restrict__ vs,
                                              int n_valid, State& st, const uint32_t (&qr)[16], float c_score, int lane) {
  const int g = lane >> 2, t4 = lane & 3;
  float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const int U = (jj & 2) * 4 + 2 * t4 + (jj & 1);
    const int up = (U & 8) | ((U ^ g) & 7);                  // (g + 8) & 7 == g & 7
    const uint4 lo = *reinterpret_cast<const uint4*>(ks + g * 256 + up * 16);
    const uint4 hi = *reinterpret_cast<const uint4*>(ks + (g + 8) * 256 + up * 16);
    mma16816<BF16>(s0, lo.x, hi.x, lo.y, hi.y, qr[4 * jj], qr[4 * jj + 1]);
    mma16816<BF16>(s1, lo.z, hi.z, lo.w, hi.w, qr[4 * jj + 2], qr[4 * jj + 3]);
  }
  float x[1][4];
  x[0][0] = (g < n_valid) ? (s0[0] + s1[0]) * c_score : -INFINITY;
  x[0][2] = (g + 8 < n_valid) ? (s0[2] + s1[2]) * c_score : -INFINITY;
  if (G4) {
    // a query group of at most 4: the lane's even column is its query, the odd one (the same query again) is not used
    move_reference_even(st, fmaxf(x[0][0], x[0][2]));
    const float o0 = (static_cast<float>(pmax_log2<16>()) - kSlack) - st.m[0];
    x[0][0] = ex2f(x[0][0] + o0); x[0][1] = 0.0f;
    x[0][2] = ex2f(x[0][2] + o0); x[0][3] = 0.0f;
  } else {
    x[0][1] = (g < n_valid) ? (s0[1] + s1[1]) * c_score : -INFINITY;
    x[0][3] = (g + 8 < n_valid) ? (s0[3] + s1[3]) * c_score : -INFINITY;
    softmax_update<1>(st, x);
  }
  uint32_t p0, p1, q0 = 0u, q1 = 0u;
  constexpr bool kLowInOddColumn = BF16 && G4;   // the odd column of a lane's query carries the low part: one product instead of two
  if (kLowInOddColumn) {
    const uint32_t h0 = pack_bf162(x[0][0], 0.0f), h2 = pack_bf162(x[0][2], 0.0f);
    const float r0 = x[0][0] - __uint_as_float(h0 << 16), r2 = x[0][2] - __uint_as_float(h2 << 16);
    p0 = movmatrix_trans(pack_bf162(__uint_as_float(h0 << 16), r0));
    p1 = movmatrix_trans(pack_bf162(__uint_as_float(h2 << 16), r2));
  } else if (BF16) {   // p~ = hi + lo, both bf16, so the weights keep ~16 bits
    const uint32_t h01 = pack_bf162(x[0][0], x[0][1]), h23 = pack_bf162(x[0][2], x[0][3]);
    const float r0 = x[0][0] - __uint_as_float(h01 << 16), r1 = x[0][1] - __uint_as_float(h01 & 0xffff0000u);
    const float r2 = x[0][2] - __uint_as_float(h23 << 16), r3 = x[0][3] - __uint_as_float(h23 & 0xffff0000u);
    p0 = movmatrix_trans(h01); p1 = movmatrix_trans(h23);
    q0 = movmatrix_trans(pack_bf162(r0, r1)); q1 = movmatrix_trans(pack_bf162(r2, r3));
  } else {
    p0 = movmatrix_trans(pack_half2(x[0][0], x[0][1]));
    p1 = movmatrix_trans(pack_half2(x[0][2], x[0][3]));
  }
  {  // running sums: a row of ones in oz row 4
    const uint32_t ones = (g == 4) ? (BF16 ? 0x3F803F80u : 0x3C003C00u) : 0u;
    mma16816<BF16>(st.oz, ones, 0u, ones, 0u, p0, p1);
    if (BF16 && !kLowInOddColumn) mma16816<BF16>(st.oz, ones, 0u, ones, 0u, q0, q1);
  }
#pragma unroll
  for (int cg = 0; cg < 4; ++cg) {
    // channels 32cg + 4g .. +3 of token rows 2t4, 2t4+1, 2t4+8, 2t4+9
    const int U = 4 * cg + (g >> 1);
    uint2 w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = 2 * t4 + (i & 1) + 8 * (i >> 1);
      const int up = (U & 8) | ((U ^ row) & 7);
      w[i] = *reinterpret_cast<const uint2*>(vs + row * 256 + up * 16 + (g & 1) * 8);
    }
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const uint32_t w0 = hf ? w[0].y : w[0].x, w1 = hf ? w[1].y : w[1].x;
      const uint32_t w2 = hf ? w[2].y : w[2].x, w3 = hf ? w[3].y : w[3].x;
      const uint32_t a0 = __byte_perm(w0, w1, 0x5410), a1 = __byte_perm(w0, w1, 0x7632);
      const uint32_t a2 = __byte_perm(w2, w3, 0x5410), a3 = __byte_perm(w2, w3, 0x7632);
      mma16816<BF16>(st.acc[2 * cg + hf], a0, a1, a2, a3, p0, p1);
      if (BF16 && !kLowInOddColumn) mma16816<BF16>(st.acc[2 * cg + hf], a0, a1, a2, a3, q0, q1);
    }
  }
}

struct SplitRange { int lo[4], hi[4]; };

// Split `split` of n_splits takes the same share of EVERY pool, so all CTAs of a (sequence,
// kv head) stream the same mix of widths: they finish together whatever a tile of each
// width costs, and the demand on HBM is even over the launch.
__device__ __forceinline__ SplitRange split_range(const int32_t* cnt_in, const long long* capacity,
                                                  int tiles_per_chunk, int split, int n_splits) {
  SplitRange r;
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    // never walk past a pool's end, whatever the table says
    const long long cnt = min(static_cast<long long>(max(cnt_in[w], 0)), capacity[w]);
    const long long n = cnt * tiles_per_chunk;
    r.lo[w] = static_cast<int>(n * split / n_splits);
    r.hi[w] = static_cast<int>(n * (split + 1) / n_splits);
  }
  return r;
}

// per-warp pipeline bookkeeping
struct Pipe {
  uint32_t ring;        // shared address of this warp's ring
  uint32_t bars;        // shared address of its 6 mbarriers
  uint32_t parity;      // bit s = parity to wait for on stage s
  bool ok;
};

// Stream `n_units` units of `unit_bytes` (each made of `pieces` bulk copies) through the ring.
// UNIT_BYTES / STAGES are compile-time; src(u, piece) gives each piece's global address.
// expect_tx + one bulk copy, executed by the whole warp without a branch: only the lane with `on` set acts
__device__ __forceinline__ void issue_copy(bool on, uint32_t bar, uint32_t dst, const void* src, uint32_t bytes, bool expect,
                                           uint32_t expect_bytes) {
  asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 p, %4, 0;\nsetp.ne.b32 q, %5, 0;\n"
               "@q mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %6;\n"
               "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%1], [%2], %3, [%0];\n}\n"
               ::"r"(bar), "r"(dst), "l"(src), "r"(bytes), "r"(on ? 1 : 0), "r"((on && expect) ? 1 : 0), "r"(expect_bytes) : "memory");
}

template <int STAGES, int STAGE_BYTES, int PIECES, typename SrcFn, typename ConsumeFn>
__device__ __forceinline__ void stream_units(Pipe& pp, int n_units, int lane, SrcFn src, ConsumeFn consume,
                                             const uint8_t* ring_generic, uint32_t last_unit_bytes = STAGE_BYTES) {
  if (n_units <= 0 || !pp.ok) return;
  // issued by the whole warp, predicated on lane 0 and on the unit's existence (no divergent branch)
  auto issue = [&](int u, bool on) {     // the last unit of the stream may be shorter
    const uint32_t bytes = (u == n_units - 1) ? last_unit_bytes : STAGE_BYTES;
    const uint32_t piece_bytes = bytes / PIECES;
    const int s = u % STAGES;
    const uint32_t bar = pp.bars + 8 * s;
#pragma unroll
    for (int p = 0; p < PIECES; ++p)
      issue_copy(on, bar, pp.ring + s * STAGE_BYTES + p * piece_bytes, src(on ? u : 0, p), piece_bytes, p == 0, bytes);
  };
  {
    const int pre = n_units < STAGES ? n_units : STAGES;
    for (int u = 0; u < pre; ++u) issue(u, lane == 0);
  }
  for (int u = 0; u < n_units; ++u) {
    const int s = u % STAGES;
    if (!mbar_wait_bounded(pp.bars + 8 * s, (pp.parity >> s) & 1u)) {
      // give the copies still in flight into this ring one more bounded wait each, so that none can
      // land after the ring has been handed on (the merge reuses it) or the CTA has exited
      for (int k = u; k < n_units && k < u + STAGES; ++k)
        mbar_wait_bounded(pp.bars + 8 * (k % STAGES), (pp.parity >> (k % STAGES)) & 1u, kWaitCycles >> 4);
      pp.ok = false;
      return;
    }
    pp.parity ^= (1u << s);
    consume(ring_generic + s * STAGE_BYTES, u);
    __syncwarp();
    issue(u + STAGES, lane == 0 && u + STAGES < n_units);
  }
}

__device__ __forceinline__ void load_qraw_rawset(uint32_t (&qr)[16], const uint16_t* qsrc, int g, int t4) {
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const int U = (jj & 2) * 4 + 2 * t4 + (jj & 1);
    const uint4 v = *reinterpret_cast<const uint4*>(qsrc + g * kHeadDim + 8 * U);
    qr[4 * jj] = v.x; qr[4 * jj + 1] = v.y; qr[4 * jj + 2] = v.z; qr[4 * jj + 3] = v.w;
  }
}

template <bool BF16, bool G4>
__global__ void __launch_bounds__(kThreads, 2)
decode_mma_kernel(Dims dm, CacheView cv, const uint16_t* __restrict__ q, int layer, float scale,
                  float* __restrict__ ws_o, float* __restrict__ ws_ml, int* __restrict__ arrived,
                  float* __restrict__ out, int n_splits, const uint16_t* __restrict__ k_new,
                  const uint16_t* __restrict__ v_new) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* rings = smem;                                              // kWarps * kRingBytes
  uint16_t* q_in = reinterpret_cast<uint16_t*>(smem + kWarps * kRingBytes);        // [8][128] input dtype
  uint16_t* q_h = q_in + 8 * kHeadDim;                                             // [8][128] fp16
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kWarps * kRingBytes + 2 * kQBytes);

  // Let a dependent launch (the next decode call, if its caller allowed the overlap) take the SM
  // slots this grid frees while its slowest CTAs are still running.
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int G = dm.n_q_heads / dm.n_kv_heads;

  // Every warp finds, for each of the 8 query rows, the power of two 2^e > max |q| (the same
  // values in all threads), then the CTA writes q (input dtype, for the 16-bit tiles) and
  // q' = q * 2^-e as fp16 (for the quantised tiles) to shared memory.
  int q_exp[8];
#pragma unroll
  for (int qi = 0; qi < 8; ++qi) {
    const int qs = G4 ? (qi >> 1) : qi;                       // G4: rows 2q and 2q + 1 both hold query q
    float mx = 0.0f;
    if (qs < G) {
      const uint2 raw4 = *reinterpret_cast<const uint2*>(q + (static_cast<long long>(b) * dm.n_q_heads + h * G + qs) * kHeadDim + 4 * lane);
      const uint32_t rw[2] = {raw4.x, raw4.y};
#pragma unroll
      for (int k = 0; k < 4; ++k)
        mx = fmaxf(mx, fabsf(load16_as_float(static_cast<uint16_t>(rw[k >> 1] >> (16 * (k & 1))), BF16 ? MOQAE_DTYPE_BF16 : MOQAE_DTYPE_FP16)));
    }
#pragma unroll
    for (int o = 1; o <= 16; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    // mx = f * 2^e with f in [1, 2): biased exponent field - 126 gives |q| < 2^e; zero rows take 0
    const int e = mx > 0.0f ? static_cast<int>((__float_as_uint(mx) >> 23) & 0xffu) - 126 : 0;
    q_exp[qi] = max(-24, min(e, 40));
  }
  for (int i = threadIdx.x; i < 8 * kHeadDim; i += kThreads) {
    const int qi = i / kHeadDim, c = i % kHeadDim;
    uint16_t raw = 0;
    const int qs = G4 ? (qi >> 1) : qi;
    if (qs < G) raw = q[(static_cast<long long>(b) * dm.n_q_heads + h * G + qs) * kHeadDim + c];
    q_in[i] = raw;
    int e = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) e = (k == qi) ? q_exp[k] : e;
    const float f = load16_as_float(raw, BF16 ? MOQAE_DTYPE_BF16 : MOQAE_DTYPE_FP16);
    q_h[i] = __half_as_ushort(__float2half_rn(f * __uint_as_float(static_cast<uint32_t>(127 - e) << 23)));
  }
  Pipe pp;
  pp.ring = smem_u32(rings + warp * kRingBytes);
  pp.bars = smem_u32(bars + warp * 6);
  pp.parity = 0u;
  pp.ok = true;
  if (lane == 0) {
    for (int s = 0; s < 6; ++s) mbar_init(pp.bars + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();

  const int group = layer / dm.rs_group;
  const int32_t* cnt = cv.count + (static_cast<long long>(group) * dm.n_tseq + table_row(dm, b, h)) * 4;
  const int tpc = tiles_per_chunk_of(dm.chunk);
  const int n_valid = tile_tokens_of(dm.chunk);      // token positions of a tile that hold tokens
  const SplitRange rg = split_range(cnt, cv.capacity, tpc, split, n_splits);

  State st;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt)
#pragma unroll
    for (int i = 0; i < 4; ++i) st.acc[mt][i] = 0.0f;
#pragma unroll
  for (int i = 0; i < 4; ++i) st.oz[i] = 0.0f;
  st.m[0] = st.m[1] = -INFINITY;

  const float log2e = 1.4426950408889634f;
  const float c_bias = scale * log2e;
  LaneConst lc;                                    // scores of quantised tiles carry 2^-24 * 2^-e
  {
    int e0 = 0, e1 = 0, eg = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      e0 = (k == 2 * t4) ? q_exp[k] : e0;
      e1 = (k == 2 * t4 + 1) ? q_exp[k] : e1;
      eg = (k == g) ? q_exp[k] : eg;
    }
    lc.cs[0] = c_bias * __uint_as_float(static_cast<uint32_t>(127 + 24 + e0) << 23);
    lc.cs[1] = c_bias * __uint_as_float(static_cast<uint32_t>(127 + 24 + e1) << 23);
    lc.cbg = c_bias * __uint_as_float(static_cast<uint32_t>(127 + eg) << 23);
  }
  const uint8_t* my_ring = rings + warp * kRingBytes;

  uint32_t qb[16], qc[16];
  // the CTA's tiles, pool after pool, are dealt to its warps round robin: `dealt` tiles so far
  int dealt = 0;

  // ---- quantised phases
  {
    // 2-bit tiles are only 3 KiB: they are fetched in pairs of neighbours (6 KiB per copy, 3 stages),
    // because the copy engine's cost per request, not HBM, bounds small copies
    const int n_tiles = rg.hi[0] - rg.lo[0];
    const int n_pairs = (n_tiles + 1) / 2;
    const int first = (warp + kWarps - dealt % kWarps) % kWarps;
    const int n = first < n_pairs ? (n_pairs - first + kWarps - 1) / kWarps : 0;
    if (n > 0) {
      const uint8_t* stream = slot_ptr(cv, dm, 0, layer, b, h, 0) + static_cast<long long>(rg.lo[0]) * 3072;
      const bool mine_is_last = (first + (n - 1) * kWarps) == n_pairs - 1;
      const uint32_t last_bytes = (mine_is_last && (n_tiles & 1)) ? 3072u : 6144u;
      phase_scale<2>(st, true);
      load_q_phase<2>(qb, qc, q_h, g, t4);
      stream_units<3, 6144, 1>(pp, n, lane,
          [&](int u, int) { return stream + static_cast<long long>(first + u * kWarps) * 6144; },
          [&](const uint8_t* tiles, int u) {
            if (u < n - 1 || last_bytes == 6144u) process_qunit<2, 2, G4>(tiles, st, qc, qb, lc, lane, n_valid);
            else process_qunit<2, 1, G4>(tiles, st, qc, qb, lc, lane, n_valid);
          }, my_ring, last_bytes);
      phase_scale<2>(st, false);
    }
    dealt += n_pairs;
  }
  {
    const int first = rg.lo[1] + (warp + kWarps - dealt % kWarps) % kWarps;
    const int n = first < rg.hi[1] ? (rg.hi[1] - first + kWarps - 1) / kWarps : 0;
    if (n > 0) {
      const uint8_t* stream = slot_ptr(cv, dm, 1, layer, b, h, 0);
      phase_scale<4>(st, true);
      load_q_phase<4>(qb, qc, q_h, g, t4);
      stream_units<3, 5120, 1>(pp, n, lane,
          [&](int u, int) { return stream + static_cast<long long>(first + u * kWarps) * 5120; },
          [&](const uint8_t* tile, int) { process_qunit<4, 1, G4>(tile, st, qc, qb, lc, lane, n_valid); }, my_ring);
      phase_scale<4>(st, false);
    }
    dealt += rg.hi[1] - rg.lo[1];
  }
  {
    const int first = rg.lo[2] + (warp + kWarps - dealt % kWarps) % kWarps;
    const int n = first < rg.hi[2] ? (rg.hi[2] - first + kWarps - 1) / kWarps : 0;
    if (n > 0) {
      const uint8_t* stream = slot_ptr(cv, dm, 2, layer, b, h, 0);
      phase_scale<8>(st, true);
      load_q_phase<8>(qb, qc, q_h, g, t4);
      stream_units<2, 9216, 1>(pp, n, lane,
          [&](int u, int) { return stream + static_cast<long long>(first + u * kWarps) * 9216; },
          [&](const uint8_t* tile, int) { process_qunit<8, 1, G4>(tile, st, qc, qb, lc, lane, n_valid); }, my_ring);
      phase_scale<8>(st, false);
    }
    dealt += rg.hi[2] - rg.lo[2];
  }
  // ---- 16-bit tiles: units of 16 tokens (4 KiB of key rows + 4 KiB of value rows)
  uint32_t qr[16];
  load_qraw_rawset(qr, q_in, g, t4);
  {
    const int first = rg.lo[3] + (warp + kWarps - dealt % kWarps) % kWarps;
    const int n = first < rg.hi[3] ? (rg.hi[3] - first + kWarps - 1) / kWarps : 0;
    if (n > 0) {
      const uint8_t* stream = slot_ptr(cv, dm, 3, layer, b, h, 0);
      phase_scale<16>(st, true);
      stream_units<2, 8192, 2>(pp, 2 * n, lane,
          [&](int u, int piece) {
            return stream + static_cast<long long>(first + (u >> 1) * kWarps) * kRawTileBytes + piece * 8192 + (u & 1) * 4096;
          },
          [&](const uint8_t* stg, int u) {
            const int nv = min(16, n_valid - 16 * (u & 1));   // a short chunk's tile: rows past n_valid are padding
            if (nv > 0) process_raw16<BF16, G4>(stg, stg + 4096, nv, st, qr, c_bias, lane);
          }, my_ring);
      phase_scale<16>(st, false);
    }
  }
  // ---- 16-bit tail (last split, warp 0): rows are staged by hand, swizzled, zero padded
  if (split == n_splits - 1 && warp == 0 && pp.ok) {
    // k_new / v_new (optional): the current token's own rows, attended to as the row after the tail
    // without being in the cache yet
    const int tail_rows = cv.tail_len[layer * dm.batch + b];
    const int len = tail_rows + (k_new ? 1 : 0);
    const long long nbase = (static_cast<long long>(b) * dm.n_kv_heads + h) * kHeadDim;
    const long long tbase = ((static_cast<long long>(layer) * dm.batch + b) * dm.n_kv_heads + h) * dm.tail_capacity * kHeadDim;
    uint8_t* stg = rings;    // warp 0's ring; all its bulk copies have completed
    phase_scale<16>(st, true);
    for (int t0 = 0; t0 < len; t0 += 16) {
      const int nv = min(16, len - t0);
      __syncwarp();
      for (int i = lane; i < 16 * 16; i += 32) {          // 16 rows x 16 units
        const int row = i >> 4, U = i & 15;
        const int up = (U & 8) | ((U ^ row) & 7);
        uint4 kv = make_uint4(0u, 0u, 0u, 0u), vv = kv;
        if (t0 + row < tail_rows) {
          kv = *reinterpret_cast<const uint4*>(cv.tail_k + tbase + static_cast<long long>(t0 + row) * kHeadDim + 8 * U);
          vv = *reinterpret_cast<const uint4*>(cv.tail_v + tbase + static_cast<long long>(t0 + row) * kHeadDim + 8 * U);
        } else if (row < nv) {
          kv = *reinterpret_cast<const uint4*>(k_new + nbase + 8 * U);
          vv = *reinterpret_cast<const uint4*>(v_new + nbase + 8 * U);
        }
        *reinterpret_cast<uint4*>(stg + row * 256 + up * 16) = kv;
        *reinterpret_cast<uint4*>(stg + 4096 + row * 256 + up * 16) = vv;
      }
      __syncwarp();
      process_raw16<BF16, G4>(stg, stg + 4096, nv, st, qr, c_bias, lane);
    }
    phase_scale<16>(st, false);
  }
  const bool timed_out = !pp.ok;

  // ---- merge: lanes -> warp -> CTA -> split partial
  __syncthreads();                       // every warp is done with its ring
  float* red_o = reinterpret_cast<float*>(smem);                 // [kWarps][8 q][128 c]
  float* red_ml = red_o + kWarps * 8 * kHeadDim;                 // [kWarps][8 q][2]
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    const int cg = mt >> 1;
    const float z0 = __shfl_sync(0xffffffffu, st.oz[0], cg * 4 + t4);
    const float z1 = __shfl_sync(0xffffffffu, st.oz[1], cg * 4 + t4);
    const int ch = 32 * cg + 4 * g + 2 * (mt & 1);
    float* o0 = red_o + (warp * 8 + 2 * t4) * kHeadDim;
    float* o1 = o0 + kHeadDim;
    if (G4) {   // the odd column holds what 16-bit tiles added through the low parts of their weights (zero otherwise)
      o0[ch] = (st.acc[mt][0] + z0) + (st.acc[mt][1] + z1); o0[ch + 1] = (st.acc[mt][2] + z0) + (st.acc[mt][3] + z1);
    } else {
      o0[ch] = st.acc[mt][0] + z0; o0[ch + 1] = st.acc[mt][2] + z0;
      o1[ch] = st.acc[mt][1] + z1; o1[ch + 1] = st.acc[mt][3] + z1;
    }
  }
  if (g == 4) {                          // this lane's oz row holds the sums
    red_ml[(warp * 8 + 2 * t4) * 2] = st.m[0]; red_ml[(warp * 8 + 2 * t4) * 2 + 1] = G4 ? st.oz[0] + st.oz[1] : st.oz[0];
    if (!G4) { red_ml[(warp * 8 + 2 * t4 + 1) * 2] = st.m[1]; red_ml[(warp * 8 + 2 * t4 + 1) * 2 + 1] = st.oz[1]; }
  }
  __syncthreads();
  // Everything up to here only read the caller's inputs and worked in registers and shared memory.
  // Workspace and output are shared with the previous kernel on the stream when this launch was
  // allowed to overlap it: wait for that kernel to complete (returns at once otherwise).
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  if (timed_out && lane == 0) set_status(cv.status, MOQAE_ERR_TIMEOUT, blockIdx.x, warp);
  for (int i = threadIdx.x; i < G * kHeadDim; i += kThreads) {
    const int qi = i / kHeadDim, c = i % kHeadDim;
    const int col = G4 ? 2 * qi : qi;      // fragment column (row of the reduction buffers) that holds query qi
    float m = -INFINITY;
#pragma unroll
    for (int wv = 0; wv < kWarps; ++wv) m = fmaxf(m, red_ml[(wv * 8 + col) * 2]);
    float l = 0.0f, o = 0.0f;
#pragma unroll
    for (int wv = 0; wv < kWarps; ++wv) {
      const float mw = red_ml[(wv * 8 + col) * 2];
      const float f = (mw == -INFINITY) ? 0.0f : ex2f(mw - m);
      l += red_ml[(wv * 8 + col) * 2 + 1] * f;
      o += red_o[(wv * 8 + col) * kHeadDim + c] * f;
    }
    const long long row = (static_cast<long long>(b) * dm.n_q_heads + h * G + qi) * n_splits + split;
    ws_o[row * kHeadDim + c] = o;
    if (c == 0) { ws_ml[row * 2] = m; ws_ml[row * 2 + 1] = l; }
  }

  // ---- split combine by the CTA that finishes last for this (sequence, kv head): no second
  // launch and nobody waits - a counter tells each CTA whether all the others are already done
  __shared__ int s_last;
  __threadfence();                       // this CTA's partials are visible device-wide ...
  __syncthreads();
  // atomicInc wraps: the arrival that finds n_splits - 1 is the last one and leaves the counter at 0
  // for the next launch, so no launch has to clear it
  if (threadIdx.x == 0)
    s_last = (atomicInc(reinterpret_cast<unsigned int*>(&arrived[b * dm.n_kv_heads + h]), static_cast<unsigned int>(n_splits - 1)) ==
              static_cast<unsigned int>(n_splits - 1)) ? 1 : 0;
  __syncthreads();                       // ... before its arrival is counted
  if (!s_last) return;
  __threadfence();
  for (int i = threadIdx.x; i < G * kHeadDim; i += kThreads) {
    const int qi = i / kHeadDim, c = i % kHeadDim;
    const long long row0 = (static_cast<long long>(b) * dm.n_q_heads + h * G + qi) * n_splits;
    // out = sum_s o_s 2^(m_s - m*) / sum_s l_s 2^(m_s - m*); partials of other CTAs: read through L2
    float m = -INFINITY;
    for (int sp = 0; sp < n_splits; ++sp) m = fmaxf(m, __ldcg(ws_ml + (row0 + sp) * 2));
    float l = 0.0f, o = 0.0f;
    for (int sp = 0; sp < n_splits; ++sp) {
      const float ms = __ldcg(ws_ml + (row0 + sp) * 2);
      const float f = (ms == -INFINITY) ? 0.0f : ex2f(ms - m);
      l += __ldcg(ws_ml + (row0 + sp) * 2 + 1) * f;
      o += __ldcg(ws_o + (row0 + sp) * kHeadDim + c) * f;
    }
    out[(static_cast<long long>(b) * dm.n_q_heads + h * G + qi) * kHeadDim + c] = l > 0.0f ? o / l : 0.0f;
  }
}

}  // namespace

int decode_mma_ctas_per_sm() { return 2; }

cudaError_t launch_decode_mma(const Dims& dm, const CacheView& cv, const void* q, int layer, float scale,
                              float* ws_o, float* ws_ml, int* arrived, float* out, int n_splits, bool overlap_previous,
                              const void* k_new, const void* v_new, cudaStream_t st) {
  const size_t smem = static_cast<size_t>(kWarps) * kRingBytes + 2 * kQBytes + kWarps * 6 * 8;
  const bool g4 = dm.n_q_heads / dm.n_kv_heads <= 4;
  auto launch = [&](auto kernel) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(n_splits, dm.n_kv_heads, dm.batch);
    lc.blockDim = dim3(kThreads, 1, 1);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    // programmatic dependent launch: this grid's CTAs may become resident as soon as every CTA of
    // the previous kernel on the stream has started and SM slots free up; the kernel itself waits
    // for that kernel's completion (griddepcontrol.wait) before its first global write
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = overlap_previous ? 1 : 0;
    return cudaLaunchKernelEx(&lc, kernel, dm, cv, static_cast<const uint16_t*>(q), layer, scale, ws_o, ws_ml, arrived, out,
                              n_splits, static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new));
  };
  cudaError_t e;
  if (dm.dtype == MOQAE_DTYPE_BF16) e = g4 ? launch(decode_mma_kernel<true, true>) : launch(decode_mma_kernel<true, false>);
  else e = g4 ? launch(decode_mma_kernel<false, true>) : launch(decode_mma_kernel<false, false>);
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

}  // namespace moqae
