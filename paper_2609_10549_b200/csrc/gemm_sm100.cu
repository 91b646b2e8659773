// Table-driven persistent BF16 GEMM for sm_100a (tcgen05 + TMEM + TMA).
//
// One launch executes a list of "blocks" (contiguous output row ranges, for the
// fused operators one block = one entry of the ring chunk schedule, Section
// III-B) as 128x256 tiles.  Tile t of the launch is handled by CTA
// (t mod gridDim.x); because the blocks are listed in schedule order, tiles are
// issued to the SMs in schedule order.
//
//   AllGather+GEMM: the A tile of a block is TMA-loaded straight from the shard
//     of the rank that owns the partition (gather by address);
//   GEMM+ReduceScatter, segmented K: the k-loop of a tile runs over the P ranks'
//     K slices in ring order into one TMEM accumulator (in-kernel reduction);
//   GEMM+ReduceScatter, ring RMW: the epilogue adds the partial tile into the
//     owner's rows in ring order (ordered read-modify-write).
//
// Warp roles (192 threads, 1 CTA per SM): warp 0 = TMA producer (one lane),
// warp 1 = tensor-memory allocation + MMA issue (one lane), warps 2..5 =
// epilogue (warp w reads TMEM lanes 32*(w%4)..+31).  A 4-stage shared-memory
// ring feeds the tensor core; two 256-column TMEM accumulators let the
// epilogue of tile i overlap the main loop of tile i+1.  Every wait is bounded.
#include "internal.h"
#include "ptx_sm100.cuh"

namespace compass {

using namespace ptx;

namespace {

constexpr int kStages = 4;
constexpr int kThreads = 192;
constexpr int kAStageBytes = BM * BK * 2;     // 16 KB
constexpr int kBStageBytes = BN * BK * 2;     // 32 KB
constexpr int kStageBytes = kAStageBytes + kBStageBytes;
constexpr uint32_t kTmemCols = 512;           // two BN-column FP32 accumulators
constexpr int kEpilogueWarps = 4;

struct Control {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort;
};

constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + size_t(kStages) * kStageBytes + sizeof(Control);

__device__ __forceinline__ void report_timeout(const GemmParams& p, Control* ctl, int site, int tile) {
  *reinterpret_cast<volatile int*>(&ctl->abort) = 1;
  if (atomicCAS(&p.status->code, 0, int(COMPASS_ERR_TIMEOUT)) == 0) {
    p.status->detail = site;
    p.status->block_idx = int(blockIdx.x);
    p.status->tile = tile;
  }
}

// Wait for an mbarrier phase, giving up after p.wait_limit_us or when another
// role of this CTA has already given up.
__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, Control* ctl, const GemmParams& p, int site,
                                             int tile) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  const uint64_t limit = uint64_t(p.wait_limit_us) * 1000ull;
  for (uint32_t spins = 1; spins < (1u << 30); ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins & 0xFF) == 0) {
      if (*reinterpret_cast<volatile int*>(&ctl->abort)) return false;
      if (globaltimer_ns() - t0 > limit) break;
    }
  }
  report_timeout(p, ctl, site, tile);
  return false;
}

struct TileCoord {
  int blk, mt, nt;
};
__device__ __forceinline__ TileCoord decode_tile(const GemmParams& p, int t) {
  const int per_block = p.tiles_m * p.tiles_n;
  TileCoord c;
  c.blk = t / per_block;
  const int w = t - c.blk * per_block;
  c.mt = w / p.tiles_n;
  c.nt = w - c.mt * p.tiles_n;
  return c;
}

__global__ void __launch_bounds__(kThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);   // 128B-swizzle tiles need 1024-byte alignment
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kStages * kAStageBytes;
  Control* ctl = reinterpret_cast<Control*>(smem + kStages * kStageBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->acc_full[b], 1);
      mbar_init(&ctl->acc_empty[b], kEpilogueWarps);
    }
    mbar_init(&ctl->drain, 1);
    ctl->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&ctl->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;

  const int total_kb = p.n_seg * p.kb_per_seg;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t issued = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < p.total_tiles; t += gridDim.x) {
        const TileCoord tc = decode_tile(p, t);
        const BlockDesc& b = p.blocks[tc.blk];
        const int a_row = b.a_row0 + tc.mt * BM;
        const int b_row = tc.nt * BN;
        for (int seg = 0; ok && seg < p.n_seg; ++seg) {
          const int am = (p.n_seg > 1) ? p.seg_rank[tc.blk][seg] : b.a_map;
          const int bm = (p.n_seg > 1) ? am : b.b_map;
          for (int kb = 0; kb < p.kb_per_seg; ++kb) {
            if (!wait_bounded(&ctl->empty[stage], phase ^ 1u, ctl, p, WAIT_SMEM_EMPTY, t)) {
              ok = false;
              break;
            }
            mbar_arrive_expect_tx(&ctl->full[stage], kStageBytes);
            tma_load_2d(smem_a + stage * kAStageBytes, &p.a_maps[am], &ctl->full[stage], kb * BK, a_row);
            tma_load_2d(smem_b + stage * kBStageBytes, &p.b_maps[bm], &ctl->full[stage], kb * BK, b_row);
            ++issued;
            if (++stage == kStages) {
              stage = 0;
              phase ^= 1u;
            }
          }
        }
      }
      // Do not leave the CTA while bulk copies may still be writing shared
      // memory: the most recent fill of every stage must have landed.
      const uint32_t outstanding = issued < uint32_t(kStages) ? issued : uint32_t(kStages);
      for (uint32_t i = 0; i < outstanding; ++i) {
        stage = (stage == 0) ? kStages - 1 : stage - 1;
        if (stage == kStages - 1) phase ^= 1u;
        if (!wait_bounded(&ctl->full[stage], phase, ctl, p, WAIT_DRAIN, -1)) break;
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(BM, BN);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < p.total_tiles; t += gridDim.x, ++it) {
        const uint32_t buf = it & 1u;
        const uint32_t acc_phase = (it >> 1) & 1u;
        if (!wait_bounded(&ctl->acc_empty[buf], acc_phase ^ 1u, ctl, p, WAIT_ACC_EMPTY, t)) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + buf * BN;
        int kb_in_seg = 0;
        for (int kb = 0; kb < total_kb; ++kb) {
          if (!wait_bounded(&ctl->full[stage], phase, ctl, p, WAIT_SMEM_FULL, t)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint64_t da = umma_smem_desc_sw128(smem_u32(smem_a + stage * kAStageBytes));
          const uint64_t db = umma_smem_desc_sw128(smem_u32(smem_b + stage * kBStageBytes));
          const int ksteps = (kb_in_seg == p.kb_per_seg - 1) ? p.tail_ksteps : BK / UMMA_K;
          for (int k = 0; k < ksteps; ++k) {
            // advance 16 elements = 32 bytes inside the 128-byte swizzle row: +2 in the address field
            umma_bf16(d_tmem, da + uint64_t(k * 2), db + uint64_t(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&ctl->empty[stage]);       // stage reusable once these MMAs have read it
          if (++kb_in_seg == p.kb_per_seg) kb_in_seg = 0;
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (ok) umma_commit(&ctl->acc_full[buf]);   // accumulator complete
      }
      if (*reinterpret_cast<volatile int*>(&ctl->abort)) {
        // Gave up somewhere: wait for whatever the tensor core still has in
        // flight before tensor memory is released.
        umma_commit(&ctl->drain);
        wait_bounded(&ctl->drain, 0, ctl, p, WAIT_DRAIN, -2);
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;               // TMEM lanes this warp may touch
    const int row_in_tile = quarter * 32 + lane;
    uint32_t it = 0;
    for (int t = blockIdx.x; t < p.total_tiles; t += gridDim.x, ++it) {
      const uint32_t buf = it & 1u;
      const uint32_t acc_phase = (it >> 1) & 1u;
      if (!wait_bounded(&ctl->acc_full[buf], acc_phase, ctl, p, WAIT_ACC_FULL, t)) break;
      tc_fence_after_sync();
      const TileCoord tc = decode_tile(p, t);
      const BlockDesc& b = p.blocks[tc.blk];
      const int row_in_block = tc.mt * BM + row_in_tile;
      const bool row_ok = row_in_block < p.rows_per_block;
      const int ncols = min(BN, p.N - tc.nt * BN);
      const int nchunks = (ncols + 31) >> 5;
      __nv_bfloat16* orow = p.out[b.out_idx] + int64_t(b.out_row0 + row_in_block) * p.ldo + int64_t(tc.nt) * BN;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + buf * BN;
      for (int c = 0; c < nchunks; ++c) {
        uint32_t v[32];
        tmem_ld_32x32b_x32(taddr + c * 32, v);
        tmem_ld_wait();
        if (c == nchunks - 1) {
          // accumulator fully copied to registers: hand it back to the MMA warp
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&ctl->acc_empty[buf]);
        }
        if (row_ok) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            if (c * 32 + g * 8 < ncols) {
              uint4 q;
              q.x = pack_bf16x2(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1]));
              q.y = pack_bf16x2(__uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3]));
              q.z = pack_bf16x2(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5]));
              q.w = pack_bf16x2(__uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7]));
              *reinterpret_cast<uint4*>(orow + c * 32 + g * 8) = q;
            }
          }
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- host side ----------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
  }
  return fn;
}

// K-major BF16 matrix [rows x K]; box = BK columns x box_rows rows, 128-byte swizzle, zero fill outside.
bool encode_kmajor(CUtensorMap* map, const void* ptr, int64_t rows, int64_t K, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cuuint64_t(K), cuuint64_t(rows)};
  cuuint64_t strides[1] = {cuuint64_t(K) * 2};
  cuuint32_t box[2] = {cuuint32_t(BK), cuuint32_t(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

size_t gemm_smem_bytes() { return kSmemBytes; }

int launch_gemm(const GemmLaunch& L, cudaStream_t stream) {
  static thread_local GemmParams p;
  for (int i = 0; i < L.n_a; ++i)
    if (!encode_kmajor(&p.a_maps[i], L.a_ptr[i], L.a_rows, L.K, BM)) return record_cuda_error(cudaErrorUnknown);
  for (int i = 0; i < L.n_b; ++i)
    if (!encode_kmajor(&p.b_maps[i], L.b_ptr[i], L.N, L.K, BN)) return record_cuda_error(cudaErrorUnknown);
  for (int i = 0; i < L.n_out; ++i) p.out[i] = static_cast<__nv_bfloat16*>(L.out_ptr[i]);
  p.ldo = L.ldo;
  p.n_blocks = L.n_blocks;
  p.rows_per_block = L.rows_per_block;
  p.N = int32_t(L.N);
  p.n_seg = L.n_seg;
  p.kb_per_seg = int32_t((L.K + BK - 1) / BK);
  const int64_t k_tail = L.K - int64_t(p.kb_per_seg - 1) * BK;
  p.tail_ksteps = int32_t((k_tail + UMMA_K - 1) / UMMA_K);
  p.tiles_m = (L.rows_per_block + BM - 1) / BM;
  p.tiles_n = int32_t((L.N + BN - 1) / BN);
  p.total_tiles = L.n_blocks * p.tiles_m * p.tiles_n;
  p.epilogue = L.epilogue;
  p.last_step = L.last_step;
  p.wait_limit_us = 2000000u;
  p.status = L.status;
  p.tile_counters = L.tile_counters;
  for (int b = 0; b < L.n_blocks; ++b) p.blocks[b] = L.blocks[b];
  if (L.n_seg > 1)
    for (int b = 0; b < L.n_blocks; ++b)
      for (int s = 0; s < L.n_seg; ++s) p.seg_rank[b][s] = L.seg_rank[b][s];

  static int num_sms = 0;
  static bool attr_set = false;
  if (!attr_set) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemBytes));
    if (e != cudaSuccess) return record_cuda_error(e);
    attr_set = true;
  }
  if (p.total_tiles <= 0) return COMPASS_OK;
  const int grid = p.total_tiles < num_sms ? p.total_tiles : num_sms;
  gemm_kernel<<<grid, kThreads, kSmemBytes, stream>>>(p);
  count_kernel_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return record_cuda_error(e);
  return COMPASS_OK;
}

}  // namespace compass
