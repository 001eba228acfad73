// Chunk router (Section 3.2, Eq. 1 and Eq. 2; Section 3.4 routing freezing).
//
// route_score_vote_kernel: a warp scores 16 tokens at a time.  The two first-layer products
// C*W1 and C*W2 are one skinny GEMM with N = 2*M = 8 output columns, which is exactly the
// m16n8k16 tensor-core shape: A = 16 token rows x 16 channels straight from global memory,
// B = the transposed weights staged once per CTA in shared memory, float32 accumulators.
// The epilogue applies the product, SiLU, W3 and the bias, takes the per-token arg-max and
// adds the 16 choices to the chunk's histogram with integer atomics (order-independent).
// HBM-bound: every hidden row is read once.
//
// finalize_map_kernel: per sequence, chunk winner (first maximum), routing freezing,
// per-width counts and slot = rank among earlier chunks of the same width.
#include <cuda_bf16.h>

#include "common.cuh"

namespace moqae {

namespace {

constexpr int kRouteWarps = 8;
constexpr int kWPad = 32;   // elements of padding per transposed weight row (bank spread)

template <bool BF16>
__device__ __forceinline__ void mma16816(float d[4], const uint32_t a[4], uint32_t b0, uint32_t b1) {
  if (BF16) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  } else {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
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
__global__ void __launch_bounds__(kRouteWarps * 32)
route_score_vote_kernel(Dims dm, int32_t* __restrict__ votes /* [batch][max_chunks][4] of the group */,
                        const uint16_t* __restrict__ hidden, int T, const uint16_t* __restrict__ W1,
                        const uint16_t* __restrict__ W2, const float* __restrict__ W3,
                        const float* __restrict__ bias, long long n_blocks16, int first_chunk) {
  extern __shared__ __align__(16) uint16_t wt[];   // [8][d_in + kWPad], row n<4: W1[:,n]; n>=4: W2[:,n-4]
  const int D = dm.d_in;
  const int ld = D + kWPad;
  for (int i = threadIdx.x; i < D * 4; i += blockDim.x) {
    const int c = i >> 2, n = i & 3;
    wt[n * ld + c] = W1[i];
    wt[(4 + n) * ld + c] = W2 ? W2[i] : static_cast<uint16_t>(0);
  }
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int C = T / dm.chunk;
  const int blocks_per_chunk = dm.chunk / 16;
  const int routed_chunks = C - first_chunk;
  float w3[4][4], bs[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    bs[i] = bias ? bias[i] : 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) w3[i][j] = W3 ? W3[i * 4 + j] : 0.0f;
  }

  for (long long blk = static_cast<long long>(blockIdx.x) * kRouteWarps + warp; blk < n_blocks16;
       blk += static_cast<long long>(gridDim.x) * kRouteWarps) {
    const int sub = static_cast<int>(blk % blocks_per_chunk);
    long long r = blk / blocks_per_chunk;
    const int c = first_chunk + static_cast<int>(r % routed_chunks);
    const int b = static_cast<int>(r / routed_chunks);
    const long long tok0 = static_cast<long long>(b) * T + static_cast<long long>(c) * dm.chunk + sub * 16;
    const uint4* row_lo = reinterpret_cast<const uint4*>(hidden + (tok0 + g) * D) + t4;
    const uint4* row_hi = reinterpret_cast<const uint4*>(hidden + (tok0 + g + 8) * D) + t4;
    const uint16_t* wrow = wt + g * ld + 8 * t4;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    float acc2[4] = {0.f, 0.f, 0.f, 0.f};
    const int n_win = D / 32;
#pragma unroll 4
    for (int w = 0; w < n_win; ++w) {
      const uint4 lo = __ldg(row_lo + 4 * w);
      const uint4 hi = __ldg(row_hi + 4 * w);
      const uint4 bw = *reinterpret_cast<const uint4*>(wrow + 32 * w);
      const uint32_t a1[4] = {lo.x, hi.x, lo.y, hi.y};
      const uint32_t a2[4] = {lo.z, hi.z, lo.w, hi.w};
      mma16816<BF16>(acc, a1, bw.x, bw.y);
      mma16816<BF16>(acc2, a2, bw.z, bw.w);
    }
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
    int32_t* vrow = votes + (static_cast<long long>(b) * dm.max_chunks + c) * 4;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const unsigned m1 = __ballot_sync(0xffffffffu, t4 == 0 && e_lo == k);
      const unsigned m2 = __ballot_sync(0xffffffffu, t4 == 0 && e_hi == k);
      const int cnt = __popc(m1) + __popc(m2);
      if (lane == 0 && cnt) atomicAdd(vrow + k, cnt);
    }
  }
}

// One CTA per sequence.  forced_map == nullptr: winners from the vote histograms.
__global__ void __launch_bounds__(256)
finalize_map_kernel(Dims dm, CacheView cv, int group, int n_chunks, const uint8_t* __restrict__ forced_map) {
  __shared__ int s_cnt[256][4];
  const int b = blockIdx.x;
  const int tid = threadIdx.x;
  const long long base = (static_cast<long long>(group) * dm.batch + b) * dm.max_chunks;
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
    cv.count[(static_cast<long long>(group) * dm.batch + b) * 4 + tid] = run;
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 4; ++k) cnt[k] = s_cnt[tid][k];
  for (int c = c0; c < c1; ++c) {
    const int w = map[c];
    slot[c] = cnt[w]++;
  }
}

}  // namespace

cudaError_t launch_route(const Dims& dm, const CacheView& cv, const void* hidden, int T, const void* W1,
                         const void* W2, const float* W3, const float* bias, int group,
                         int32_t* votes_out, cudaStream_t st) {
  const int C = T / dm.chunk;
  const long long tbl = static_cast<long long>(group) * dm.batch * dm.max_chunks;
  int32_t* votes = cv.votes + tbl * 4;
  cudaError_t e = cudaMemsetAsync(votes, 0, sizeof(int32_t) * 4 * static_cast<size_t>(dm.batch) * dm.max_chunks, st);
  if (e != cudaSuccess) return e;
  const int first = dm.rf_first_chunk ? 1 : 0;
  const long long n_blocks16 = static_cast<long long>(dm.batch) * (C > first ? C - first : 0) * (dm.chunk / 16);
  if (n_blocks16 > 0) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const size_t smem = sizeof(uint16_t) * 8 * static_cast<size_t>(dm.d_in + kWPad);
    long long want = (n_blocks16 + kRouteWarps - 1) / kRouteWarps;
    const long long cap = static_cast<long long>(sms) * 2;
    const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
    if (dm.dtype == MOQAE_DTYPE_BF16) {
      e = cudaFuncSetAttribute(route_score_vote_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      route_score_vote_kernel<true><<<grid, kRouteWarps * 32, smem, st>>>(
          dm, votes, static_cast<const uint16_t*>(hidden), T, static_cast<const uint16_t*>(W1),
          static_cast<const uint16_t*>(W2), W3, bias, n_blocks16, first);
    } else {
      e = cudaFuncSetAttribute(route_score_vote_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      route_score_vote_kernel<false><<<grid, kRouteWarps * 32, smem, st>>>(
          dm, votes, static_cast<const uint16_t*>(hidden), T, static_cast<const uint16_t*>(W1),
          static_cast<const uint16_t*>(W2), W3, bias, n_blocks16, first);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  e = launch_finalize_map(dm, cv, group, C, nullptr, st);
  if (e != cudaSuccess) return e;
  if (votes_out && C > 0) {
    e = cudaMemcpy2DAsync(votes_out, sizeof(int32_t) * 4 * C, votes, sizeof(int32_t) * 4 * dm.max_chunks,
                          sizeof(int32_t) * 4 * C, dm.batch, cudaMemcpyDeviceToDevice, st);
  }
  return e;
}

cudaError_t launch_finalize_map(const Dims& dm, const CacheView& cv, int group, int n_chunks,
                                const uint8_t* forced_map, cudaStream_t st) {
  finalize_map_kernel<<<dm.batch, 256, 0, st>>>(dm, cv, group, n_chunks, forced_map);
  return cudaGetLastError();
}

}  // namespace moqae
