// Chunk router (Section 3.2, Eq. 1 and Eq. 2; Section 3.4 routing freezing).
//
// route_score_vote_kernel: every warp is an independent stream over 16-token blocks.  The
// hidden rows arrive through tiled TMA copies (boxes of 64 channels x 16 tokens, 128-byte
// swizzle, four boxes per pipeline stage) into the warp's own two-stage ring, so 16 KiB per
// warp are always in flight.  The two first-layer products C*W1 and C*W2 are one skinny GEMM
// with N = 2*M = 8 output columns, which is exactly the m16n8k16 tensor-core shape: A = 16
// token rows x 16 channels read with ldmatrix (conflict-free under the swizzle), B = the
// transposed weights staged once per CTA in shared memory, float32 accumulators.  The
// epilogue applies the product, SiLU, W3 and the bias, takes the per-token arg-max and adds
// the 16 choices to the chunk's histogram with integer atomics (order-independent).
// HBM-bound: every hidden row is read once.
//
// finalize_map_kernel: per sequence, chunk winner (first maximum), routing freezing,
// per-width counts and slot = rank among earlier chunks of the same width.
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace moqae {

namespace {

constexpr int kMaxRouteWarps = 8;
constexpr int kWPad = 8;             // elements of padding per transposed weight row (bank spread)
constexpr int kBoxCols = 64;         // channels per TMA box (128 bytes: the swizzle span)
constexpr int kBoxBytes = 16 * 128;  // 16 token rows
constexpr int kBoxesPerStage = 4;
constexpr int kStageBytes = kBoxesPerStage * kBoxBytes;
constexpr int kStages = 2;
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&a)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(addr));
}

template <bool BF16>
__device__ __forceinline__ void mma16816(float d[4], const uint32_t a[4], uint32_t b0, uint32_t b1) {
  if (BF16) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  } else {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  }
}

__device__ __forceinline__ float silu(float a) { return a / (1.0f + expf(-a)); }

// First index of the maximum of four values.
__device__ __forceinline__ int argmax4(float p0, float p1, float p2, float p3) {
  int e = 0;
  float m = p0;
  if (p1 > m) { m = p1; e = 1; }
  if (p2 > m) { m = p2; e = 2; }
  if (p3 > m) { m = p3; e = 3; }
  return e;
}

template <bool BF16>
__global__ void __launch_bounds__(kMaxRouteWarps * 32)
route_score_vote_kernel(Dims dm, int32_t* __restrict__ votes /* [batch][max_chunks][4] of the group */,
                        const __grid_constant__ CUtensorMap map_hidden, int T, const uint16_t* __restrict__ W1,
                        const uint16_t* __restrict__ W2, const float* __restrict__ W3,
                        const float* __restrict__ bias, long long n_blocks16, int first_chunk, int32_t* status,
                        const int32_t* __restrict__ append_after /* nullable: [batch][4] chunk counts */) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // the swizzled TMA boxes want 1024-byte alignment: round the base up (the launch adds the slack)
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const int D = dm.d_in;
  const int n_boxes = (D + kBoxCols - 1) / kBoxCols;
  const int Dpad = n_boxes * kBoxCols;
  const int ld = Dpad + kWPad;
  const int n_warps = blockDim.x >> 5;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint8_t* ring = smem + warp * (kStages * kStageBytes);
  uint16_t* wt = reinterpret_cast<uint16_t*>(smem + n_warps * (kStages * kStageBytes));   // [8][ld]: W1^T then W2^T
  uint64_t* bars = reinterpret_cast<uint64_t*>(wt + 8 * ld) + kStages * warp;
  for (int i = threadIdx.x; i < Dpad * 4; i += blockDim.x) {
    const int c = i >> 2, n = i & 3;
    wt[n * ld + c] = c < D ? W1[i] : static_cast<uint16_t>(0);
    wt[(4 + n) * ld + c] = (W2 && c < D) ? W2[i] : static_cast<uint16_t>(0);
  }
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(bars + s), 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();

  const int g = lane >> 2, t4 = lane & 3;
  const int C = T / dm.chunk;
  // The hidden rows are walked in blocks of 16 tokens.  A chunk of 16 j tokens is j blocks; with
  // chunks of 8 tokens one block holds two chunks (rows 0..7 and 8..15 vote separately).
  const bool two_chunks = dm.chunk == 8;
  const int blocks_per_chunk = two_chunks ? 1 : dm.chunk / 16;
  const int routed_chunks = C - first_chunk;
  const int blocks_per_seq = two_chunks ? (routed_chunks + 1) / 2 : routed_chunks * blocks_per_chunk;
  float w3[4][4], bs[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    bs[i] = bias ? bias[i] : 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) w3[i][j] = W3 ? W3[i * 4 + j] : 0.0f;
  }
  const int n_stages = (n_boxes + kBoxesPerStage - 1) / kBoxesPerStage;     // per 16-token block
  const long long blk0 = static_cast<long long>(blockIdx.x) * n_warps + warp;
  const long long blk_stride = static_cast<long long>(gridDim.x) * n_warps;
  const long long my_blocks = blk0 < n_blocks16 ? (n_blocks16 - blk0 + blk_stride - 1) / blk_stride : 0;
  const long long total_units = my_blocks * n_stages;                      // this warp's stream of stages

  auto block_coords = [&](long long blk, int& b, int& c, int& row) {
    const int i = static_cast<int>(blk % blocks_per_seq);
    b = static_cast<int>(blk / blocks_per_seq);
    const int sub = two_chunks ? 0 : i % blocks_per_chunk;
    c = first_chunk + (two_chunks ? 2 * i : i / blocks_per_chunk);
    // b is the table row: a sequence, or with per-head routing (sequence, kv head) = (b / H, b % H)
    row = (dm.per_head ? b / dm.n_kv_heads : b) * T + c * dm.chunk + sub * 16;
  };
  // Lane 0 issues the stages of this warp's stream in order; the cursor (block, stage, ring slot and the
  // block's coordinates) moves along with it, so the divisions of block_coords run once per block and
  // not once per stage.
  long long ib_i = 0;
  int st_i = 0, slot_i = 0, b_i = 0, c_i = 0, row_i = 0;
  if (lane == 0 && my_blocks > 0) block_coords(blk0, b_i, c_i, row_i);
  auto issue_next = [&]() {             // lane 0
    const int box0 = st_i * kBoxesPerStage;
    const int nb = min(kBoxesPerStage, n_boxes - box0);
    const uint32_t bar = smem_u32(bars + slot_i);
    mbar_expect_tx(bar, nb * kBoxBytes);
    const int head = dm.per_head ? b_i % dm.n_kv_heads : 0;   // middle coordinate: which 128-wide row of the token
    for (int i = 0; i < nb; ++i)
      tma_load_3d(smem_u32(ring + slot_i * kStageBytes + i * kBoxBytes), &map_hidden, (box0 + i) * kBoxCols, head, row_i, bar);
    slot_i = slot_i + 1 == kStages ? 0 : slot_i + 1;
    if (++st_i == n_stages) {
      st_i = 0;
      if (++ib_i < my_blocks) block_coords(blk0 + ib_i * blk_stride, b_i, c_i, row_i);
    }
  };
  if (lane == 0)
    for (long long u = 0; u < kStages && u < total_units; ++u) issue_next();

  // ldmatrix row address of this lane inside a box: matrices (rows 0-7 | 8-15) x (k 0-7 | 8-15)
  const int lm_row = (lane & 7) + ((lane >> 3) & 1) * 8;
  const int lm_half = lane >> 4;
  const uint16_t* wrow = wt + g * ld + 2 * t4;
  uint32_t parity = 0;                  // bit s: parity to wait for on stage s
  bool ok = true;
  long long u = 0;
  for (long long ib = 0; ib < my_blocks && ok; ++ib) {
    const long long blk = blk0 + ib * blk_stride;
    int b, c, row;
    block_coords(blk, b, c, row);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    float acc2[4] = {0.f, 0.f, 0.f, 0.f};
    for (int st = 0; st < n_stages; ++st, ++u) {
      const int slot = static_cast<int>(u % kStages);
      if (!mbar_wait_bounded(smem_u32(bars + slot), (parity >> slot) & 1u)) { ok = false; break; }
      parity ^= 1u << slot;
      const int box0 = st * kBoxesPerStage;
      const int nb = min(kBoxesPerStage, n_boxes - box0);
      const uint32_t stage_base = smem_u32(ring + slot * kStageBytes);
      for (int i = 0; i < nb; ++i) {
        const uint32_t box_base = stage_base + i * kBoxBytes + lm_row * 128;
        const uint16_t* wk = wrow + (box0 + i) * kBoxCols;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          uint32_t a[4];
          ldmatrix_x4(a, box_base + (((2 * kk + lm_half) ^ (lm_row & 7)) << 4));
          const uint32_t b0 = *reinterpret_cast<const uint32_t*>(wk + 16 * kk);
          const uint32_t b1 = *reinterpret_cast<const uint32_t*>(wk + 16 * kk + 8);
          mma16816<BF16>((kk & 1) ? acc2 : acc, a, b0, b1);
        }
      }
      __syncwarp();
      if (lane == 0 && u + kStages < total_units) issue_next();
    }
    if (!ok) break;
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] += acc2[i];
    // acc[0], acc[1]: token g, columns 2*t4, 2*t4+1; acc[2], acc[3]: token g+8.
    int e_lo, e_hi;
    if (W2) {
      // columns 0..3 = u, 4..7 = v: lanes t4 = 0,1 fetch v from lanes t4+2
      const float v0 = __shfl_down_sync(0xffffffffu, acc[0], 2), v1 = __shfl_down_sync(0xffffffffu, acc[1], 2);
      const float v2 = __shfl_down_sync(0xffffffffu, acc[2], 2), v3 = __shfl_down_sync(0xffffffffu, acc[3], 2);
      float pl[4] = {0.f, 0.f, 0.f, 0.f}, ph[4] = {0.f, 0.f, 0.f, 0.f};
      if (t4 < 2) {
        const float h0 = silu(acc[0] * v0), h1 = silu(acc[1] * v1);
        const float h2 = silu(acc[2] * v2), h3 = silu(acc[3] * v3);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float wa = t4 == 0 ? w3[0][k] : w3[2][k];
          const float wb = t4 == 0 ? w3[1][k] : w3[3][k];
          pl[k] = h0 * wa + h1 * wb;
          ph[k] = h2 * wa + h3 * wb;
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        pl[k] += __shfl_xor_sync(0xffffffffu, pl[k], 1);
        ph[k] += __shfl_xor_sync(0xffffffffu, ph[k], 1);
      }
      e_lo = argmax4(pl[0] + bs[0], pl[1] + bs[1], pl[2] + bs[2], pl[3] + bs[3]);
      e_hi = argmax4(ph[0] + bs[0], ph[1] + bs[1], ph[2] + bs[2], ph[3] + bs[3]);
    } else {
      // linear router: columns 0..3 are the logits; lane t4=0 holds 0,1 and lane t4=1 holds 2,3
      const float o0 = __shfl_xor_sync(0xffffffffu, acc[0], 1), o1 = __shfl_xor_sync(0xffffffffu, acc[1], 1);
      const float o2 = __shfl_xor_sync(0xffffffffu, acc[2], 1), o3 = __shfl_xor_sync(0xffffffffu, acc[3], 1);
      e_lo = argmax4(acc[0] + bs[0], acc[1] + bs[1], o0 + bs[2], o1 + bs[3]);
      e_hi = argmax4(acc[2] + bs[0], acc[3] + bs[1], o2 + bs[2], o3 + bs[3]);
    }
    // prefill: the chunk's own row; flush of a full tail: the row after the sequence's last chunk
    int c_row = c;
    if (append_after) c_row = append_after[4 * b] + append_after[4 * b + 1] + append_after[4 * b + 2] + append_after[4 * b + 3];
    if (c_row >= dm.max_chunks) continue;
    int32_t* vrow = votes + (static_cast<long long>(b) * dm.max_chunks + c_row) * 4;
    // rows 8..15 of the block: the same chunk, or (chunks of 8 tokens) the next one if it exists
    const bool hi_counts = !two_chunks || (c + 1 < C && c_row + 1 < dm.max_chunks);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const unsigned m1 = __ballot_sync(0xffffffffu, t4 == 0 && e_lo == k);
      const unsigned m2 = __ballot_sync(0xffffffffu, t4 == 0 && e_hi == k);
      if (two_chunks) {
        if (lane == 0 && m1) atomicAdd(vrow + k, __popc(m1));
        if (lane == 0 && m2 && hi_counts) atomicAdd(vrow + 4 + k, __popc(m2));
      } else {
        const int cnt = __popc(m1) + __popc(m2);
        if (lane == 0 && cnt) atomicAdd(vrow + k, cnt);
      }
    }
  }
  if (!ok) {
    // a copy did not land in time: report it and give the copies in flight a last bounded chance
    if (lane == 0) set_status(status, MOQAE_ERR_TIMEOUT, blockIdx.x, warp);
    for (int s = 0; s < kStages; ++s) mbar_wait_bounded(smem_u32(bars + s), (parity >> s) & 1u);
  }
}

// One CTA per sequence.  forced_map == nullptr: winners from the vote histograms.
__global__ void __launch_bounds__(256)
finalize_map_kernel(Dims dm, CacheView cv, int group, int n_chunks, const uint8_t* __restrict__ forced_map) {
  __shared__ int s_cnt[256][4];
  const int b = blockIdx.x;
  const int tid = threadIdx.x;
  const long long base = (static_cast<long long>(group) * dm.n_tseq + b) * dm.max_chunks;
  uint8_t* map = cv.map + base;
  int32_t* slot = cv.slot + base;
  const int32_t* votes = cv.votes + base * 4;
  const int per = (n_chunks + 255) / 256;
  const int c0 = min(n_chunks, tid * per), c1 = min(n_chunks, c0 + per);
  int cnt[4] = {0, 0, 0, 0};
  for (int c = c0; c < c1; ++c) {
    int w;
    if (forced_map) {
      w = forced_map[static_cast<long long>(b) * n_chunks + c];
      if (w > 3) w = 3;
    } else if (c == 0 && dm.rf_first_chunk) {
      w = 3;
    } else {
      const int4 v = *reinterpret_cast<const int4*>(votes + 4 * c);
      w = 0;
      int m = v.x;
      if (v.y > m) { m = v.y; w = 1; }
      if (v.z > m) { m = v.z; w = 2; }
      if (v.w > m) { m = v.w; w = 3; }
    }
    map[c] = static_cast<uint8_t>(w);
    cnt[w]++;
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) s_cnt[tid][k] = cnt[k];
  __syncthreads();
  if (tid < 4) {   // exclusive scan over the 256 thread ranges, one expert per thread
    int run = 0;
    for (int i = 0; i < 256; ++i) {
      const int v = s_cnt[i][tid];
      s_cnt[i][tid] = run;
      run += v;
    }
    cv.count[(static_cast<long long>(group) * dm.n_tseq + b) * 4 + tid] = run;
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 4; ++k) cnt[k] = s_cnt[tid][k];
  for (int c = c0; c < c1; ++c) {
    const int w = map[c];
    slot[c] = cnt[w]++;
  }
}

// flush step 1: clear the vote row the new chunk of every sequence will use
__global__ void flush_prepare_kernel(Dims dm, int32_t* __restrict__ votes, const int32_t* __restrict__ count_g) {
  const int b = blockIdx.x;
  const int c = count_g[4 * b] + count_g[4 * b + 1] + count_g[4 * b + 2] + count_g[4 * b + 3];
  if (threadIdx.x < 4 && c < dm.max_chunks) votes[(static_cast<long long>(b) * dm.max_chunks + c) * 4 + threadIdx.x] = 0;
}

// flush step 3: winner of the new chunk, its slot, tables.  A sequence takes part only if the
// tail of the group's first layer is exactly full.  The map entry carries bit 7 until the
// chunk's rows have been packed (flush_reset_kernel clears it), which is how the packing
// kernels know that the sequence is being flushed.
__global__ void flush_finalize_kernel(Dims dm, CacheView cv, int group) {
  if (threadIdx.x != 0) return;
  const int b = blockIdx.x;
  const int layer0 = group * dm.rs_group;
  if (cv.tail_len[layer0 * dm.batch + b] != dm.chunk) return;
  int32_t* count = cv.count + (static_cast<long long>(group) * dm.batch + b) * 4;
  const int c = count[0] + count[1] + count[2] + count[3];
  if (c >= dm.max_chunks) { set_status(cv.status, MOQAE_ERR_POOL_FULL, -3, c); return; }
  const long long base = (static_cast<long long>(group) * dm.batch + b) * dm.max_chunks;
  const int32_t* v = cv.votes + (base + c) * 4;
  int w = 0, m = v[0];
  if (v[1] > m) { m = v[1]; w = 1; }
  if (v[2] > m) { m = v[2]; w = 2; }
  if (v[3] > m) { m = v[3]; w = 3; }
  if (c == 0 && dm.rf_first_chunk) w = 3;                  // routing freezing: the first chunk stays 16-bit
  const int slot = count[w];
  if (slot >= cv.capacity[w]) { set_status(cv.status, MOQAE_ERR_POOL_FULL, w, slot); return; }
  cv.map[base + c] = static_cast<uint8_t>(w | 0x80);
  cv.slot[base + c] = slot;
  count[w] = slot + 1;
}

}  // namespace

// Launch the scoring + voting kernel over hidden [batch][T][d_in]: chunks first..C-1 of every sequence.
static cudaError_t launch_score_vote(const Dims& dm, const CacheView& cv, const void* hidden, int T, int first,
                                     const void* W1, const void* W2, const float* W3, const float* bias,
                                     int32_t* votes, const int32_t* append_after, cudaStream_t st) {
  const int C = T / dm.chunk;
  const int routed = C > first ? C - first : 0;
  const long long n_blocks16 = static_cast<long long>(dm.n_tseq) * (dm.chunk == 8 ? (routed + 1) / 2 : routed * (dm.chunk / 16));
  if (n_blocks16 <= 0) return cudaSuccess;
  int dev = 0, sms = 148, smem_max = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  // [batch*T][d_in] 16-bit tensor, boxes of 64 channels x 16 tokens, 128-byte swizzle
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap map;
  // viewed as [batch * T tokens][rows per token][d_in]: one row per token, or with per-head routing
  // the token's n_kv_heads rows of 128 channels; a box is 16 tokens of ONE such row
  const cuuint64_t per_tok = dm.per_head ? dm.n_kv_heads : 1;
  const cuuint64_t gdim[3] = {static_cast<cuuint64_t>(dm.d_in), per_tok, static_cast<cuuint64_t>(dm.batch) * T};
  const cuuint64_t gstride[2] = {static_cast<cuuint64_t>(dm.d_in) * 2, static_cast<cuuint64_t>(dm.d_in) * 2 * per_tok};
  const cuuint32_t box[3] = {kBoxCols, 1, 16};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void*>(hidden), gdim, gstride, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  const int n_boxes = (dm.d_in + kBoxCols - 1) / kBoxCols;
  const size_t wt_bytes = sizeof(uint16_t) * 8 * static_cast<size_t>(n_boxes * kBoxCols + kWPad);
  // as many warps (each with its own ring) as fit beside the weights, one CTA per SM
  int warps = kMaxRouteWarps;
  auto smem_for = [&](int w) { return static_cast<size_t>(w) * kStages * kStageBytes + wt_bytes + 8 * kStages * w + 1024; };
  while (warps > 1 && smem_for(warps) > static_cast<size_t>(smem_max)) --warps;
  if (smem_for(warps) > static_cast<size_t>(smem_max)) return cudaErrorInvalidConfiguration;
  const size_t smem = smem_for(warps);
  long long want = (n_blocks16 + warps - 1) / warps;
  const unsigned grid = static_cast<unsigned>(want < sms ? want : sms);
  cudaError_t e;
  if (dm.dtype == MOQAE_DTYPE_BF16) {
    e = cudaFuncSetAttribute(route_score_vote_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    route_score_vote_kernel<true><<<grid, warps * 32, smem, st>>>(
        dm, votes, map, T, static_cast<const uint16_t*>(W1), static_cast<const uint16_t*>(W2), W3, bias,
        n_blocks16, first, cv.status, append_after);
  } else {
    e = cudaFuncSetAttribute(route_score_vote_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    route_score_vote_kernel<false><<<grid, warps * 32, smem, st>>>(
        dm, votes, map, T, static_cast<const uint16_t*>(W1), static_cast<const uint16_t*>(W2), W3, bias,
        n_blocks16, first, cv.status, append_after);
  }
  return cudaGetLastError();
}

cudaError_t launch_route(const Dims& dm, const CacheView& cv, const void* hidden, int T, const void* W1,
                         const void* W2, const float* W3, const float* bias, int group,
                         int32_t* votes_out, cudaStream_t st) {
  const int C = T / dm.chunk;
  const long long tbl = static_cast<long long>(group) * dm.n_tseq * dm.max_chunks;
  int32_t* votes = cv.votes + tbl * 4;
  cudaError_t e = cudaMemsetAsync(votes, 0, sizeof(int32_t) * 4 * static_cast<size_t>(dm.n_tseq) * dm.max_chunks, st);
  if (e != cudaSuccess) return e;
  e = launch_score_vote(dm, cv, hidden, T, dm.rf_first_chunk ? 1 : 0, W1, W2, W3, bias, votes, nullptr, st);
  if (e != cudaSuccess) return e;
  e = launch_finalize_map(dm, cv, group, C, nullptr, st);
  if (e != cudaSuccess) return e;
  if (votes_out && C > 0) {
    e = cudaMemcpy2DAsync(votes_out, sizeof(int32_t) * 4 * C, votes, sizeof(int32_t) * 4 * dm.max_chunks,
                          sizeof(int32_t) * 4 * C, dm.n_tseq, cudaMemcpyDeviceToDevice, st);
  }
  return e;
}

// ---- flush of a full 16-bit tail: the tail's tokens become one more routed chunk -------------
cudaError_t launch_flush_route(const Dims& dm, const CacheView& cv, const void* hidden_tail, const void* W1,
                               const void* W2, const float* W3, const float* bias, int group, cudaStream_t st) {
  const long long tbl = static_cast<long long>(group) * dm.batch * dm.max_chunks;
  int32_t* votes = cv.votes + tbl * 4;
  const int32_t* count_g = cv.count + static_cast<long long>(group) * dm.batch * 4;
  flush_prepare_kernel<<<dm.batch, 32, 0, st>>>(dm, votes, count_g);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  // the tail is one chunk per sequence: T = chunk, nothing frozen here (chunk 0 is handled below)
  e = launch_score_vote(dm, cv, hidden_tail, dm.chunk, 0, W1, W2, W3, bias, votes, count_g, st);
  if (e != cudaSuccess) return e;
  flush_finalize_kernel<<<dm.batch, 32, 0, st>>>(dm, cv, group);
  return cudaGetLastError();
}

cudaError_t launch_finalize_map(const Dims& dm, const CacheView& cv, int group, int n_chunks,
                                const uint8_t* forced_map, cudaStream_t st) {
  finalize_map_kernel<<<dm.n_tseq, 256, 0, st>>>(dm, cv, group, n_chunks, forced_map);
  return cudaGetLastError();
}

}  // namespace moqae
