// Structures shared between the host-side planner and the kernels.
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/compass.h"

namespace compass {

constexpr int kMaxP = COMPASS_MAX_P;
constexpr int kMaxBlocks = 2 * kMaxP * kMaxP;   // rings * P * P schedule entries
constexpr int kMaxSegBlocks = 2 * kMaxP;        // blocks of a segmented-K launch (rings * P partitions)

// Tile shape of the GEMM kernel (one CTA computes BM x BN of the output).
constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;          // 64 BF16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;

// Device status block at the start of a workspace.
struct StatusBlock {
  int32_t code;      // compass_status
  int32_t detail;    // which wait gave up (WaitSite) and where
  int32_t block_idx;
  int32_t tile;
  // written by CTA 0 of every GEMM launch that uses this block: SM cycles and nanoseconds from its start to its end
  unsigned long long kernel_cycles;
  unsigned long long kernel_ns;
};

// Element-wise function between the accumulator and the store (values of COMPASS_ACT_*).
enum ActivationMode : int32_t { ACT_NONE = 0, ACT_GELU_TANH = 1, ACT_SWIGLU = 2 };

enum WaitSite : int32_t {
  WAIT_NONE = 0,
  WAIT_SMEM_EMPTY = 1,     // TMA producer waiting for a free pipeline stage
  WAIT_SMEM_FULL = 2,      // MMA issuer waiting for operands
  WAIT_ACC_EMPTY = 3,      // MMA issuer waiting for a free accumulator
  WAIT_ACC_FULL = 4,       // epilogue waiting for an accumulator
  WAIT_DRAIN = 5,          // teardown waiting for outstanding work
  WAIT_TILE_COUNTER = 6,   // ring read-modify-write waiting for the previous contributor
  WAIT_READY_FLAG = 7,     // TMA producer waiting for a pushed partition to arrive
};

// A block is a contiguous range of output rows handled as tiles_m x tiles_n
// tiles.  For the fused kernels one block = one schedule entry.
struct BlockDesc {
  int32_t a_row0;     // first row read from the A tensor(s)
  int32_t out_row0;   // first row written in the output tensor
  uint8_t a_map;      // index of the A tensor map (single-segment launches)
  uint8_t b_map;      // index of the B tensor map (single-segment launches)
  uint8_t out_idx;    // index of the output pointer
  uint8_t step;       // schedule step (ring read-modify-write: contributor index)
  uint8_t part;       // schedule partition id
  uint8_t seg_stride; // strided segments (GemmParams.seg_strided): segment s reads tensor (a_map + s * seg_stride) mod n_ranks
  uint16_t flag1;     // 1 + index of the readiness flag the block's A rows wait for (0 = always ready)
};

enum GemmMode : int32_t {
  GEMM_MODE_AUTO = 0,     // CTA pairs when a block has at least 256 rows
  GEMM_MODE_SINGLE = 1,   // one CTA per 128x256 tile
  GEMM_MODE_PAIR = 2,     // two CTAs per 256x256 tile
  GEMM_MODE_MIXED = 3,    // CTA pairs: 512x256 tiles for the full waves, 256x256 for the tail
};

enum EpilogueMode : int32_t {
  EPI_STORE = 0,      // round to BF16 and store
  EPI_RING_RMW = 1,   // ordered accumulate into the output in ring order
  EPI_RING_RMW_F32 = 2,   // the same with the running sum in FP32 scratch; the last contributor writes the BF16 output
};

constexpr int kMaxAMaps = 2 * kMaxP;   // shards plus, for the push variant, the per-rank gather buffers

struct GemmParams {
  CUtensorMap a_maps[kMaxAMaps];
  CUtensorMap b_maps[kMaxP];
  CUtensorMap b_maps_q[kMaxP];   // the same B tensors with boxes of 64 rows (256x128 tiles: 64 B rows per CTA)
  __nv_bfloat16* out[kMaxP];
  uint8_t* ring_scratch;   // ring read-modify-write: running sums, one 128 x 256 fragment after the other in the order
                           // of the tile counters, each in the order its epilogue warps' lanes hold it
  int64_t ldo;             // output row pitch in elements
  int32_t n_blocks;
  int32_t rows_per_block;
  int32_t N;               // output columns
  int32_t n_seg;           // K segments accumulated into one tile (1, or P for segmented-K reduce)
  int32_t kb_per_seg;      // k-stages per segment (last one may be partial)
  int32_t tail_ksteps;     // UMMA_K steps in the last k-stage of a segment
  // Blocks of fewer than 256 rows that read the same B tensor are tiled together: `group` consecutive blocks,
  // each padded to `sub_pad` rows (a multiple of 128), form one virtual block of group * sub_pad rows, so that
  // every 128-row fragment of a tile lies inside ONE block and a CTA pair can work on two blocks at once.
  // group = 1 and sub_pad >= rows_per_block for ordinary blocks.
  int32_t group;
  int32_t sub_pad;
  int32_t vrows;           // rows of a virtual block: group * sub_pad
  int32_t frags_m;         // 128-row fragments per block: ceil(rows_per_block / 128)
  int32_t tiles_m, tiles_n; // tiles per virtual block
  int32_t total_tiles;
  // mixed-tile pair kernel: tiles [0, n_big) are 512x256, tiles [n_big, n_small_end) 256x256 (two per remaining
  // 512x256 slot), tiles [n_small_end, total_tiles) 256x128 (four per slot)
  int32_t n_big;
  int32_t n_small_end;
  int32_t big_tiles_m;     // 512-row tiles per block
  int32_t h_last;          // 256-row halves of a block's last 512-row slot that hold rows: 2, or 1 when at most 256 rows are left
  int32_t kb_big;          // 64-wide k-stages per segment of a big tile
  int32_t tail_big;        // UMMA_K steps in its last stage
  int32_t epilogue;        // EpilogueMode
  int32_t last_step;       // ring RMW: step index of the final contributor (P-1)
  uint32_t wait_limit_us;  // bound of every device-side wait
  int32_t a_hint, b_hint;  // L2 eviction priority of the A / B tile loads (ptx::L2Hint)
  int32_t prefetch_stages; // how many k-stages ahead of the shared-memory loads operands are prefetched into L2 (0 = off)
  int32_t b_mn_major;      // 1: the B tensors are stored [K][N] (N contiguous); 0: [N][K]
  int32_t activation;      // ActivationMode applied to the FP32 accumulator before the BF16 store (plain-store epilogue only)
  int32_t skew;            // 512x256 tiles: stages at each end of a tile in which accumulator 0 runs ahead of accumulator 1 (0..4)
  StatusBlock* status;
  int32_t* tile_counters;  // ring RMW only
  const uint32_t* flags;   // readiness flags (push variant), else nullptr
  uint32_t flag_token;     // a flag is up once it holds a value >= this
  uint8_t seg_rank[kMaxSegBlocks][kMaxP];   // segmented-K: tensor index of segment s of block b
  int32_t seg_strided;     // 1: the segments' tensors follow BlockDesc.a_map and seg_stride instead of seg_rank
  int32_t n_ranks;
  BlockDesc blocks[kMaxBlocks];
};

// Host-side description of a GEMM launch before tensor maps are encoded.
struct GemmLaunch {
  const void* a_ptr[kMaxAMaps];
  int64_t a_map_rows[kMaxAMaps] = {};   // rows of A tensor i; 0 = a_rows
  const void* b_ptr[kMaxP];
  void* out_ptr[kMaxP];
  void* ring_scratch = nullptr;   // running sums of the ring read-modify-write epilogues (one fragment per tile counter)
  int n_a = 0, n_b = 0, n_out = 0;
  int64_t a_rows = 0;      // rows of every A tensor
  int64_t K = 0;           // columns (contraction length) of every A and B tensor
  int64_t N = 0;           // rows of every B tensor = output columns
  int64_t ldo = 0;
  int n_seg = 1;
  int rows_per_block = 0;
  int share_run = 1;       // blocks come in aligned runs of this many consecutive blocks that read the same B tensor
  int epilogue = EPI_STORE;
  int mode = GEMM_MODE_AUTO;
  int a_hint = 0;   // ptx::L2Hint of the A loads
  int b_hint = 2;   // weight tiles: evict last (measured 1-2 % shorter kernels than the default priority)
  int prefetch_stages = 0;
  int activation = 0;   // ActivationMode
  int b_mn_major = 0;   // 1: B tensors are [K][N]
  int skew = 3;     // 512x256 tiles: stages at each end of a tile with accumulator 0 ahead of accumulator 1 (measured: 3 of 0..4)
  uint32_t wait_limit_us = 0;   // 0 = default bound of the device-side waits
  int last_step = 0;
  int n_blocks = 0;
  BlockDesc blocks[kMaxBlocks];
  uint8_t seg_rank[kMaxSegBlocks][kMaxP];
  bool seg_strided = false;   // segments by BlockDesc.a_map / seg_stride (grouped ring read-modify-write) instead of seg_rank
  int n_ranks = 0;
  StatusBlock* status = nullptr;
  int32_t* tile_counters = nullptr;
  const uint32_t* flags = nullptr;
  uint32_t flag_token = 0;
};

// How a launch is cut into tiles, decided on the host from the block list and the number of co-resident CTA pairs.
struct TilePlan {
  int32_t pair;          // 1: clusters of two CTAs (256-row tiles); 0: single CTAs (128-row tiles)
  int32_t mixed;         // 1: the mixed-tile kernel (512x256 / 256x256 / 256x128 tiles), plain-store epilogue
  int32_t group;         // consecutive blocks tiled together (blocks below 256 rows that share a B tensor)
  int32_t sub_pad;       // rows of a block rounded up to a multiple of 128
  int32_t vrows;         // rows of a virtual block that are cut into tiles
  int32_t n_vblocks;
  int32_t tiles_m, tiles_n;
  int32_t big_tiles_m;   // 512-row slots per virtual block (mixed only)
  int32_t h_last;        // 256-row halves of a block's last slot that hold rows (mixed only)
  int32_t n_big, n_small, n_quarter;   // tiles of 512x256, 256x256 (or 128x256 when pair == 0), 256x128
  int32_t total_tiles;
};

// gemm_sm100.cu
TilePlan plan_tiles(const GemmLaunch& launch, int max_pairs);
int launch_gemm(const GemmLaunch& launch, cudaStream_t stream);
size_t gemm_smem_bytes();
void tensor_map_cache_stats(uint64_t* hits, uint64_t* misses);
int gemm_tile_rows(int mode, int rows_per_block);   // rows of one scheduling tile: 256 (CTA pair) or 128

// aux_kernels.cu
int launch_reduce_partials(const void* const* partial, int P, void* const* out, int64_t m, int64_t N,
                           int64_t slice_begin, int64_t slice_rows, cudaStream_t stream);

int launch_gather_slices(const void* const* shard, void* const* gather, int P, int64_t m, int64_t K, int64_t slice_begin,
                         int64_t slice_rows, cudaStream_t stream);

// api.cu
int record_cuda_error(cudaError_t e);
void count_kernel_launch();
uint32_t default_wait_limit_us();   // 0 = built-in default

// schedule.cpp
int build_schedule(int op, int P, int rings, int64_t M, compass_sched_entry* out);   // out has rings*P*P slots
int validate_schedule_args(int op, int P, int rings, int64_t M);

}  // namespace compass
