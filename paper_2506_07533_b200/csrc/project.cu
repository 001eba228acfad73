// Fused producer: the K and V projections of one layer with the quantiser as their epilogue.
//
// Section 3.1 of the paper: once the router has fixed the widths of a block's chunks, the chunks
// are quantised with them and the block goes on with its computation.  The keys and values that
// get quantised are the products of the block's hidden states with its key / value weights; here
// those products never travel to HBM as 16-bit rows.  One kernel computes
//     K = hidden Wk^T,  V = hidden Wv^T          (hidden [B][T][d_in], Wk / Wv [Hkv * 128][d_in])
// on the 5th-generation tensor cores (tcgen05.mma, fp32 accumulators in tensor memory), rounds
// the accumulators to the 16-bit input dtype (what a separate projection kernel would have
// stored), and runs the quantise + bit-pack path of moqae_quantize_kv on them tile by tile,
// writing pool slots (or the 16-bit tail) directly.
//
// Work unit: 128 tokens of one sequence x one kv head = an accumulator of 128 lanes x 256
// columns (K channels 0..127 | V channels 0..127), i.e. four storage tiles of keys and of values.
// Roles of the 6 warps of a persistent CTA (one per SM), meeting only on mbarriers with bounded
// waits:
//   warp 0   one thread issues the TMA copies of a 3-stage ring: per 64-wide slice of d_in a
//            128 x 64 box of hidden rows and two 128 x 64 boxes of Wk / Wv rows, 128-byte swizzle;
//   warp 1   one thread issues tcgen05.mma (M 128, N 256, K 16) from those tiles into one of two
//            accumulator buffers, so the products of the next unit run while the epilogue
//            works on the previous one;
//   warps 2..5   epilogue: warp w owns tensor-memory lanes 32 (w mod 4) .. + 31 = the 32 tokens of
//            one storage tile; it reads its rows with tcgen05.ld, rounds them, lays them out as
//            32 rows of 256 bytes in shared memory and hands them to the same encoder the
//            stand-alone quantise kernel uses; the finished tile leaves with one bulk store.
// No TMA load uses cluster multicast.
#include <cstring>

#include <cuda_bf16.h>

#include "ptx.cuh"
#include "quant_encode.cuh"

namespace moqae {

namespace {

constexpr int kBM = 128;                        // tokens per unit
constexpr int kBK = 64;                         // d_in slice per stage: 64 elements = one 128-byte swizzle row
constexpr int kPStages = 3;
constexpr int kABytes = kBM * kBK * 2;          // 16 KiB
constexpr int kBBytes = 2 * kHeadDim * kBK * 2; // 32 KiB: Wk rows, then Wv rows
constexpr int kPStageBytes = kABytes + kBBytes;
constexpr int kRowsBytes = 8192;                // 32 rows x 256 B
constexpr int kTileOutBytes = 9216;             // largest quantised tile
constexpr int kPrmBytes2 = 2048;
constexpr int kEpiBytes = kRowsBytes + kTileOutBytes + kPrmBytes2;
constexpr int kEpiWarps = 4;
constexpr int kProjThreads = (2 + kEpiWarps) * 32;
constexpr int kTmemCols = 512;                  // two accumulators of 256 columns
constexpr long long kProjWait = 1ll << 31;      // about a second of SM cycles

enum { PB_FULL = 0, PB_EMPTY = kPStages, PB_ACC_FULL = 2 * kPStages, PB_ACC_EMPTY = 2 * kPStages + 2, PB_COUNT = 2 * kPStages + 4 };

// Shared-memory matrix descriptor of a K-major operand tile in the 128-byte swizzled layout TMA
// writes: rows of 128 bytes (64 elements), 1 KiB between groups of 8 rows; start address, leading
// and stride byte offsets in units of 16 bytes, descriptor version 1 (bit 46), layout type 2
// (128-byte swizzle, bits 61..63).
__device__ __forceinline__ uint64_t desc_sw128_kmajor(uint32_t saddr) {
  return static_cast<uint64_t>((saddr >> 4) & 0x3fffu) | (static_cast<uint64_t>(16u >> 4) << 16) |
         (static_cast<uint64_t>(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// D (tensor memory) = / += A B, both operands in shared memory, one CTA
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
               ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit_to(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
// 32 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_load32(uint32_t (&r)[32], uint32_t taddr) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
template <bool BF16> __device__ __forceinline__ uint32_t round_pair(uint32_t a_bits, uint32_t b_bits) {
  const float a = __uint_as_float(a_bits), b = __uint_as_float(b_bits);
  if (BF16) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
  }
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Instruction descriptor of kind::f16: fp32 accumulator (bit 4), A and B formats (bits 7..9 and
// 10..12: 0 = fp16, 1 = bf16), both operands K-major, N >> 3 at bit 17, M >> 4 at bit 24.
template <bool BF16> __host__ __device__ constexpr uint32_t proj_idesc() {
  return (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
}

struct ProjArgs {
  int T, layer, d_in;
  int m_tiles;             // ceil(T / 128)
  long long n_units;       // batch * m_tiles * n_kv_heads
  uint16_t* dbg_k;         // optional [batch][T][n_kv_heads][128] rounded K rows (parity tests); may be null
  uint16_t* dbg_v;
};

template <bool BF16>
__global__ void __launch_bounds__(kProjThreads, 1)
project_quantize_kernel(Dims dm, CacheView cv, const __grid_constant__ CUtensorMap map_h,
                        const __grid_constant__ CUtensorMap map_wk, const __grid_constant__ CUtensorMap map_wv,
                        ProjArgs pa) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);     // swizzled tiles want 1 KiB alignment
  uint8_t* stages = smem;
  uint8_t* epi = stages + kPStages * kPStageBytes;
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(epi + kEpiWarps * kEpiBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + PB_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bar_mem);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = dm.n_kv_heads;
  const int n_kb = pa.d_in / kBK;

  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < PB_COUNT; ++i) mbar_init(bar(i), i >= PB_ACC_EMPTY ? kEpiWarps : 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  // the tail length of every sequence is a function of T alone
  if (blockIdx.x == 0 && tid < dm.batch) {
    const int r = pa.T - (pa.T / dm.chunk) * dm.chunk;
    if (r > dm.tail_capacity) set_status(cv.status, MOQAE_ERR_POOL_FULL, -1, r);
    cv.tail_len[pa.layer * dm.batch + tid] = min(r, dm.tail_capacity);
  }
  tc_before_sync();
  __syncthreads();
  tc_after_sync();
  const uint32_t tmem = *tmem_slot;

  // bounded wait on barrier i for its n-th completion (n = 0, 1, ..); a timeout aborts every role
  auto wait = [&](int i, uint32_t n) {
    if (*abort_flag) return false;
    if (mbar_wait_bounded(bar(i), n & 1u, kProjWait)) return true;
    *abort_flag = 1;
    if (lane == 0) set_status(cv.status, MOQAE_ERR_TIMEOUT, blockIdx.x, i);
    return false;
  };

  if (warp == 0) {
    // ================= TMA producer (one thread) =================
    if (lane == 0) {
      uint32_t it = 0;                                   // stage uses so far
      for (long long u = blockIdx.x; u < pa.n_units; u += gridDim.x) {
        const int h = static_cast<int>(u % H);
        const long long x = u / H;
        const int mt = static_cast<int>(x % pa.m_tiles), b = static_cast<int>(x / pa.m_tiles);
        bool ok = true;
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int st = it % kPStages;
          if (it >= kPStages) ok = wait(PB_EMPTY + st, it / kPStages - 1);
          if (!ok) break;
          uint8_t* sA = stages + st * kPStageBytes;
          mbar_expect_tx(bar(PB_FULL + st), kPStageBytes);
          tma_load_3d(smem_u32(sA), &map_h, kb * kBK, mt * kBM, b, bar(PB_FULL + st));
          tma_load_2d(smem_u32(sA + kABytes), &map_wk, kb * kBK, h * kHeadDim, bar(PB_FULL + st));
          tma_load_2d(smem_u32(sA + kABytes + kBBytes / 2), &map_wv, kb * kBK, h * kHeadDim, bar(PB_FULL + st));
        }
        if (!ok) break;
      }
      if (*abort_flag) {
        // copies may still be in flight into the ring: give each stage one more bounded wait
        for (int st = 0; st < kPStages; ++st) {
          mbar_wait_bounded(bar(PB_FULL + st), 0, kProjWait >> 6);
          mbar_wait_bounded(bar(PB_FULL + st), 1, kProjWait >> 6);
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issue (one thread) =================
    if (lane == 0) {
      uint32_t it = 0, n_unit = 0;
      for (long long u = blockIdx.x; u < pa.n_units; u += gridDim.x, ++n_unit) {
        const int buf = n_unit & 1;
        bool ok = true;
        if (n_unit >= 2) ok = wait(PB_ACC_EMPTY + buf, n_unit / 2 - 1);     // the epilogue has read this accumulator
        if (!ok) break;
        tc_after_sync();
        const uint32_t d = tmem + buf * 256;
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int st = it % kPStages;
          ok = wait(PB_FULL + st, it / kPStages);
          if (!ok) break;
          tc_after_sync();
          const uint32_t sA = smem_u32(stages + st * kPStageBytes);
          const uint64_t ad = desc_sw128_kmajor(sA), bd = desc_sw128_kmajor(sA + kABytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)               // a K step of 16 elements = 32 bytes inside the swizzled row
            umma_ss(d, ad + 2 * k, bd + 2 * k, proj_idesc<BF16>(), (kb | k) != 0);
          umma_commit_to(bar(PB_EMPTY + st));              // the stage is free once these products have read it
        }
        if (!ok) break;
        umma_commit_to(bar(PB_ACC_FULL + buf));
      }
    }
  } else {
    // ================= epilogue: 32 tokens (one storage tile) per warp =================
    const int ew = warp - 2;
    const int quarter = warp & 3;                          // the tensor-memory lanes this warp may read
    uint8_t* rows = epi + ew * kEpiBytes;
    uint8_t* out = rows + kRowsBytes;
    float4* prm = reinterpret_cast<float4*>(out + kTileOutBytes);
    const int tpc = dm.chunk / kTileTokens;
    const int C = pa.T / dm.chunk;
    const int group = pa.layer / dm.rs_group;
    bool store_pending = false;
    uint32_t n_unit = 0;
    for (long long u = blockIdx.x; u < pa.n_units; u += gridDim.x, ++n_unit) {
      const int h = static_cast<int>(u % H);
      const long long x = u / H;
      const int mt = static_cast<int>(x % pa.m_tiles), b = static_cast<int>(x / pa.m_tiles);
      const int buf = n_unit & 1;
      if (!wait(PB_ACC_FULL + buf, n_unit / 2)) break;
      tc_after_sync();
      const int t0 = mt * kBM + quarter * kTileTokens;     // first token of this warp's rows
      const int n_valid = min(kTileTokens, pa.T - t0);     // <= 0: nothing of this tile exists
      // where the tile goes
      int w = -1;
      uint8_t* tile = nullptr;
      if (n_valid > 0 && t0 < C * dm.chunk) {
        const int c = t0 / dm.chunk, j = (t0 % dm.chunk) / kTileTokens;
        const long long tbl = (static_cast<long long>(group) * dm.batch + b) * dm.max_chunks + c;
        w = cv.map[tbl];
        const int slot = cv.slot[tbl];
        long long cap = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) cap = (w == k) ? cv.capacity[k] : cap;
        if (w > 3 || slot < 0 || slot >= cap) {
          if (lane == 0) set_status(cv.status, MOQAE_ERR_POOL_FULL, w, slot);
          w = -1;
        } else {
          uint8_t* pool = cv.pool[0];
#pragma unroll
          for (int k = 1; k < 4; ++k) pool = (w == k) ? cv.pool[k] : pool;
          const long long idx = ((static_cast<long long>(pa.layer) * dm.batch + b) * H + h) * cap + slot;
          tile = pool + (idx * tpc + j) * tile_bytes_of_expert(w);
        }
      }
      const bool is_tail = n_valid > 0 && t0 >= C * dm.chunk;
#pragma unroll 1
      for (int which = 0; which < 2; ++which) {
        // accumulator rows -> 32 rows of 256 bytes in the input dtype (lane = token)
        if (which == 0 && store_pending) {                 // the previous tile's bulk store must have read `out`
          if (lane == 0) bulk_store_wait_read();
          store_pending = false;
        }
        __syncwarp();
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t r[32];
          tmem_load32(r, tmem + ((quarter * 32u) << 16) + buf * 256 + which * 128 + cc * 32);
          uint4* dst = reinterpret_cast<uint4*>(rows + lane * 256 + cc * 64);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(round_pair<BF16>(r[8 * i], r[8 * i + 1]), round_pair<BF16>(r[8 * i + 2], r[8 * i + 3]),
                                round_pair<BF16>(r[8 * i + 4], r[8 * i + 5]), round_pair<BF16>(r[8 * i + 6], r[8 * i + 7]));
        }
        if (which == 1) {                                  // both halves are out of tensor memory
          tc_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(PB_ACC_EMPTY + buf));
        }
        __syncwarp();
        if (n_valid <= 0) continue;
        uint16_t* dbg = which ? pa.dbg_v : pa.dbg_k;
        if (dbg) {
          for (int i = lane; i < n_valid * 16; i += 32) {
            const int row = i >> 4, U = i & 15;
            *reinterpret_cast<uint4*>(dbg + ((static_cast<long long>(b) * pa.T + t0 + row) * H + h) * kHeadDim + 8 * U) =
                *reinterpret_cast<const uint4*>(rows + row * 256 + U * 16);
          }
        }
        if (is_tail) {
          uint16_t* tl = which ? cv.tail_v : cv.tail_k;
          const int r0 = t0 - C * dm.chunk;
          const long long base = ((static_cast<long long>(pa.layer) * dm.batch + b) * H + h) * dm.tail_capacity;
          for (int i = lane; i < n_valid * 16; i += 32) {
            const int row = i >> 4, U = i & 15;
            if (r0 + row < dm.tail_capacity)
              *reinterpret_cast<uint4*>(tl + (base + r0 + row) * kHeadDim + 8 * U) = *reinterpret_cast<const uint4*>(rows + row * 256 + U * 16);
          }
        } else if (w == 3) {
          copy_raw_rows(rows, tile + which * 8192, lane);
        } else if (w >= 0) {
          if (which == 0) {
            if (w == 0) encode_keys<2, BF16>(rows, out, lane);
            else if (w == 1) encode_keys<4, BF16>(rows, out, lane);
            else encode_keys<8, BF16>(rows, out, lane);
          } else {
            if (w == 0) encode_values<2, BF16>(rows, out, prm, lane);
            else if (w == 1) encode_values<4, BF16>(rows, out, prm, lane);
            else encode_values<8, BF16>(rows, out, prm, lane);
            fence_async_smem();                            // generic-proxy writes to `out` -> visible to the bulk store
            __syncwarp();
            if (lane == 0) bulk_store(tile, smem_u32(out), tile_bytes_of_expert(w));
            store_pending = true;
          }
        }
        __syncwarp();
      }
    }
    if (lane == 0) bulk_store_wait_all();
  }
  tc_before_sync();
  __syncthreads();
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// [outer][rows][cols] 16-bit tensor (outer may be 1), boxes of 64 columns x 128 rows, 128-byte swizzle
bool make_operand_map(CUtensorMap* m, const void* base, long long cols, long long rows, long long outer) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t gdim[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(outer)};
  const cuuint64_t gstride[2] = {static_cast<cuuint64_t>(cols) * 2, static_cast<cuuint64_t>(cols) * static_cast<cuuint64_t>(rows) * 2};
  const cuuint32_t box[3] = {kBK, kBM, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const int rank = outer > 0 ? 3 : 2;
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT16, rank, const_cast<void*>(base), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_project_quantize(const Dims& dm, const CacheView& cv, const void* hidden, const void* Wk, const void* Wv,
                                    int T, int layer, void* dbg_k, void* dbg_v, cudaStream_t st) {
  if (T <= 0) {
    // nothing to project: only the tail lengths are defined (zero)
    return cudaMemsetAsync(cv.tail_len + static_cast<long long>(layer) * dm.batch, 0, sizeof(int32_t) * dm.batch, st);
  }
  CUtensorMap mh, mk, mv;
  memset(&mh, 0, sizeof(mh));
  memset(&mk, 0, sizeof(mk));
  memset(&mv, 0, sizeof(mv));
  const long long n_out = static_cast<long long>(dm.n_kv_heads) * kHeadDim;
  if (!make_operand_map(&mh, hidden, dm.d_in, T, dm.batch) || !make_operand_map(&mk, Wk, dm.d_in, n_out, 0) ||
      !make_operand_map(&mv, Wv, dm.d_in, n_out, 0))
    return cudaErrorNotSupported;
  ProjArgs pa;
  pa.T = T;
  pa.layer = layer;
  pa.d_in = dm.d_in;
  pa.m_tiles = (T + kBM - 1) / kBM;
  pa.n_units = static_cast<long long>(dm.batch) * pa.m_tiles * dm.n_kv_heads;
  pa.dbg_k = static_cast<uint16_t*>(dbg_k);
  pa.dbg_v = static_cast<uint16_t*>(dbg_v);
  const size_t smem = 1024 + static_cast<size_t>(kPStages) * kPStageBytes + kEpiWarps * kEpiBytes + PB_COUNT * 8 + 16;
  const long long sms = sm_count_of_current_device();
  const unsigned grid = static_cast<unsigned>(pa.n_units < sms ? pa.n_units : sms);
  cudaError_t e;
  if (dm.dtype == MOQAE_DTYPE_BF16) {
    e = cudaFuncSetAttribute(project_quantize_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    project_quantize_kernel<true><<<grid, kProjThreads, smem, st>>>(dm, cv, mh, mk, mv, pa);
  } else {
    e = cudaFuncSetAttribute(project_quantize_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    project_quantize_kernel<false><<<grid, kProjThreads, smem, st>>>(dm, cv, mh, mk, mv, pa);
  }
  return cudaGetLastError();
}

}  // namespace moqae
