// Table-driven persistent BF16 GEMMs for sm_100a (tcgen05 + TMEM + TMA).
//
// One launch executes a list of "blocks" (contiguous output row ranges, for the
// fused operators one block = one entry of the ring chunk schedule, Section
// III-B).  Tile t of the launch is handled by work unit (t mod #units);
// because the blocks are listed in schedule order, tiles are issued to the SMs
// in schedule order.
//
//   AllGather+GEMM: the A tile of a block is TMA-loaded straight from the shard
//     of the rank that owns the partition (gather by address);
//   GEMM+ReduceScatter, segmented K: the k-loop of a tile runs over the P ranks'
//     K slices in ring order into one TMEM accumulator (in-kernel reduction);
//   GEMM+ReduceScatter, ring read-modify-write: every rank's partial tile is
//     added by the epilogue to the partition's running sum in ring order (the
//     sum travels through scratch memory; the owner, last, writes its rows).
//
// Three kernels share the roles and the barrier protocol:
//   gemm_mixed_kernel  clusters of two CTAs; 512x256 tiles (two accumulators per
//                      CTA sharing one B tile) for the whole waves of a launch,
//                      256x256 and 256x128 tiles for the tail; plain-store
//                      epilogue.  The default wherever CTA pairs can be used.
//   gemm_kernel<true>  clusters of two CTAs, 256x256 tiles; carries the ring
//                      read-modify-write epilogue.
//   gemm_kernel<false> one CTA per 128x256 tile; row fragments below 256 rows.
// Each has a second instantiation whose plain-store epilogue applies an
// activation (GELU-tanh, or SwiGLU on interleaved gate/up columns) to the FP32
// accumulator: the first GEMM of the MLP block (Section II-A).  All of them
// take the weight tiles either K-contiguous ([N][K]) or N-contiguous ([K][N],
// MN-major tcgen05 operand), and CTA 0 of every launch records its SM cycles
// and nanoseconds in the status block.
// In the pair kernels each CTA loads its own rows of A and its half of the B
// rows; the leader CTA issues tcgen05.mma.cta_group::2, which reads both CTAs'
// shared memory, and each CTA's tensor memory receives its rows of the
// accumulator.  Every TMA load fills the shared memory of the CTA that issues it only.
//
// Warp roles (192 threads, 1 CTA per SM): warp 0 = TMA producer (one lane),
// warp 1 = tensor-memory allocation + MMA issue (one lane), warps 2..5 =
// epilogue (warp w reads TMEM lanes 32*(w%4)..+31).  Every wait is bounded and
// reports COMPASS_ERR_TIMEOUT instead of hanging.
#include <algorithm>
#include <atomic>
#include <mutex>

#include "internal.h"
#include "ptx_sm100.cuh"

namespace compass {

using namespace ptx;

namespace {

constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;           // two BN-column FP32 accumulators
constexpr int kEpilogueWarps = 4;
constexpr int kSlots = 4;                      // pipeline barrier pairs (>= stages of every kernel below)

template <bool kPair>
struct Cfg {
  // A pipeline stage holds kAtoms k-atoms of 64 elements (one 128-byte swizzle
  // row each).  The MMA issuer pays a fixed cost per stage (barrier wait,
  // commit, loop) of a few hundred cycles during which the tensor core only has
  // the queued MMAs to work on, so a stage must carry enough of them: 8 per
  // stage keep the pipe full, 4 do not.
  static constexpr int kAtoms = kPair ? 2 : 1;
  static constexpr int kStageK = kAtoms * BK;
  static constexpr int kStages = kPair ? 3 : 4;
  static constexpr int kAAtomBytes = BM * BK * 2;                 // 128 rows of A, one atom
  static constexpr int kBRows = kPair ? BN / 2 : BN;              // rows of B this CTA loads
  static constexpr int kBAtomBytes = kBRows * BK * 2;
  static constexpr int kATileBytes = kAtoms * kAAtomBytes;
  static constexpr int kBTileBytes = kAtoms * kBAtomBytes;
  static constexpr int kStageBytes = kATileBytes + kBTileBytes;   // per CTA
  static constexpr int kTileRows = kPair ? 2 * BM : BM;           // rows of one scheduling tile
  static constexpr uint32_t kFullTxBytes = kPair ? 2 * kStageBytes : kStageBytes;
};

// An N-contiguous B tile is kept as chunks of 64 columns x 64 k-rows (what one tensor-map box of 128-byte rows holds).
constexpr int kBChunkMnBytes = 64 * BK * 2;

struct Control {
  uint64_t full[kSlots];
  uint64_t empty[kSlots];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort;
};

// epilogue staging: per epilogue warp 32 rows x 64 BF16 columns, rows padded by 16 bytes (conflict-free 16-byte accesses)
constexpr int kStageRowBytes = 64 * 2 + 16;
constexpr int kStageWarpBytes = 32 * kStageRowBytes;

template <bool kPair>
constexpr size_t smem_bytes() {
  return 1024 /*alignment slack*/ + size_t(Cfg<kPair>::kStages) * Cfg<kPair>::kStageBytes + sizeof(Control) + 16 +
         size_t(kEpilogueWarps) * kStageWarpBytes;
}

__device__ __forceinline__ void report_timeout(const GemmParams& p, Control* ctl, int site, int tile) {
  *reinterpret_cast<volatile int*>(&ctl->abort) = 1;
  if (atomicCAS(&p.status->code, 0, int(COMPASS_ERR_TIMEOUT)) == 0) {
    p.status->detail = site;
    p.status->block_idx = int(blockIdx.x);
    p.status->tile = tile;
  }
}

// Activations of the MLP block's first GEMM, on the FP32 accumulator.  exp through the fast
// exponential (relative error ~2^-21, far below the BF16 rounding that follows).
__device__ __forceinline__ float gelu_tanh_f32(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  const float t = 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * u));       // tanh(u); exp overflow gives exactly 1
  return 0.5f * x * (1.0f + t);
}
__device__ __forceinline__ float swiglu_f32(float gate, float up) {
  return __fdividef(gate, 1.0f + __expf(-gate)) * up;                     // silu(gate) * up
}

// CTA 0 records how many SM cycles and nanoseconds it ran: their ratio is the clock the
// kernel really had (under a power cap well below the nominal one).
struct ClockRecord {
  long long c0;
  uint64_t t0;
  __device__ __forceinline__ void begin() {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      c0 = clock64();
      t0 = globaltimer_ns();
    }
  }
  __device__ __forceinline__ void end(const GemmParams& p) const {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      p.status->kernel_cycles = static_cast<unsigned long long>(clock64() - c0);
      p.status->kernel_ns = globaltimer_ns() - t0;
    }
  }
};

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

// Bounded wait until a tile counter in global memory reaches `target`.
// (Waits on something another CTA or the host must provide give up after 3/4 of the limit, so that the
// status names them and not one of the barrier waits queued up behind them in the same CTA.)
__device__ __forceinline__ bool wait_counter(const int* counter, int target, Control* ctl, const GemmParams& p, int tile) {
  const uint64_t t0 = globaltimer_ns();
  const uint64_t limit = uint64_t(p.wait_limit_us) * 750ull;
  for (uint32_t spins = 0; spins < (1u << 30); ++spins) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    if ((spins & 0x3F) == 0x3F) {
      if (*reinterpret_cast<volatile int*>(&ctl->abort)) return false;
      if (globaltimer_ns() - t0 > limit) break;
    }
  }
  report_timeout(p, ctl, WAIT_TILE_COUNTER, tile);
  return false;
}

// Bounded wait until a pushed partition has arrived: its flag (written in stream order after
// the copy that fills the rows) holds the launch's token.  The rows were written by a copy
// engine and are read next through the async proxy (TMA), hence the proxy fence.
__device__ __forceinline__ bool wait_ready_flag(const GemmParams& p, const BlockDesc& b, Control* ctl, int tile) {
  if (p.flags == nullptr || b.flag1 == 0) return true;
  const uint32_t* flag = p.flags + (b.flag1 - 1);
  const uint64_t t0 = globaltimer_ns();
  const uint64_t limit = uint64_t(p.wait_limit_us) * 750ull;
  for (uint32_t spins = 0; spins < (1u << 30); ++spins) {
    uint32_t v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v >= p.flag_token) {
      asm volatile("fence.proxy.async;" ::: "memory");
      return true;
    }
    if ((spins & 0x3F) == 0x3F) {
      if (*reinterpret_cast<volatile int*>(&ctl->abort)) return false;
      if (globaltimer_ns() - t0 > limit) break;
    }
  }
  report_timeout(p, ctl, WAIT_READY_FLAG, tile);
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

// A 128-row fragment of a tile: which block it lies in and its first row inside that block.  `vblk` is the
// virtual block (p.group consecutive blocks, each padded to p.sub_pad rows), `v0` the fragment's first
// virtual row, a multiple of 128.  Fragments past the last block are mapped beyond that block's rows, where
// every row is masked.
struct Frag {
  int blk, r0;
};
__device__ __forceinline__ Frag fragment_of(const GemmParams& p, int vblk, int v0) {
  if (p.group == 1) return Frag{vblk, v0};
  int j = v0 / p.sub_pad;
  if (j >= p.group) j = p.group - 1;
  return Frag{vblk * p.group + j, v0 - j * p.sub_pad};
}

// Walks the sequence of k-stages one work unit loads: for every tile of the
// unit (t, t + n_units, ...), every K segment, every k-stage of the segment.
template <bool kPair>
struct StageIter {
  int t, step, cta_rank;
  int seg, kb;
  int blk;                   // block this CTA's 128 rows of A belong to
  int am, bm, a_row, b_row;
  __device__ StageIter(const GemmParams& p, int unit, int n_units, int rank) : t(unit), step(n_units), cta_rank(rank), seg(0), kb(0) {
    if (valid(p)) enter(p);
  }
  __device__ bool valid(const GemmParams& p) const { return t < p.total_tiles; }
  __device__ void enter(const GemmParams& p) {      // refresh what depends on (t, seg)
    const TileCoord tc = decode_tile(p, t);
    const Frag f = fragment_of(p, tc.blk, tc.mt * Cfg<kPair>::kTileRows + cta_rank * BM);
    const BlockDesc& b = p.blocks[f.blk];
    blk = f.blk;
    a_row = b.a_row0 + f.r0;
    b_row = tc.nt * BN + cta_rank * Cfg<kPair>::kBRows;
    // segmented K (blocks are never grouped): the segment's tensor from the table, or, along a ring, a stride from the lead's
    am = (p.n_seg > 1) ? (p.seg_strided ? (int(b.a_map) + seg * int(b.seg_stride)) % p.n_ranks : int(p.seg_rank[tc.blk][seg]))
                       : int(b.a_map);
    bm = (p.n_seg > 1) ? am : b.b_map;                           // the blocks of a group share their B tensor
  }
  __device__ void next(const GemmParams& p) {
    if (++kb < p.kb_per_seg) return;
    kb = 0;
    if (++seg == p.n_seg) {
      seg = 0;
      t += step;
    }
    if (valid(p)) enter(p);
  }
};

// kAct: the plain-store epilogue applies p.activation (its own instantiation, see gemm_mixed_kernel).
// kF32Sum: the ring read-modify-write epilogue keeps the running sum in FP32 instead of BF16 (again its own
// instantiation).
template <bool kPair, bool kAct, bool kF32Sum>
__global__ void __launch_bounds__(kThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
  using C = Cfg<kPair>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);   // 128B-swizzle tiles need 1024-byte alignment
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + C::kStages * C::kATileBytes;
  Control* ctl = reinterpret_cast<Control*>(smem + C::kStages * C::kStageBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = kPair ? cluster_ctarank() : 0u;    // 0 = leader of the pair
  const bool leader = cta_rank == 0;
  // work units: clusters in pair mode, CTAs otherwise
  const int unit = kPair ? int(blockIdx.x >> 1) : int(blockIdx.x);
  const int n_units = kPair ? int(gridDim.x >> 1) : int(gridDim.x);
  ClockRecord clock_record;
  clock_record.begin();

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->acc_full[b], 1);
      mbar_init(&ctl->acc_empty[b], kPair ? 2 * kEpilogueWarps : kEpilogueWarps);
    }
    mbar_init(&ctl->drain, 1);
    ctl->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    if (kPair) {
      tmem_alloc_pair(&ctl->tmem_base, kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(&ctl->tmem_base, kTmemCols);
      tmem_relinquish();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (kPair) {
    // both CTAs' barriers and tensor memory exist before either CTA signals the other
    cluster_arrive();
    cluster_wait();
  }
  tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;

  const int total_kb = p.n_seg * p.kb_per_seg;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t issued = 0;
      const uint64_t pol_a = make_l2_policy(p.a_hint);
      const uint64_t pol_b = make_l2_policy(p.b_hint);
      // `ld` walks this unit's (tile, segment, k-stage) sequence; `pf` can run
      // p.prefetch_stages ahead of it and pull the boxes into L2 only.  Off by
      // default: on B200 the prefetches compete with the loads for the same
      // request path and slow the kernel down (measured: up to 2x).
      StageIter<kPair> ld(p, unit, n_units, int(cta_rank));
      StageIter<kPair> pf(p, unit, n_units, int(cta_rank));
      for (int i = 0; i < p.prefetch_stages && pf.valid(p); ++i) pf.next(p);
      int ready_t = -1;
      while (ld.valid(p)) {
        if (ld.t != ready_t) {      // first stage of a tile: its A rows may still be on their way
          if (!wait_ready_flag(p, p.blocks[ld.blk], ctl, ld.t)) break;
          ready_t = ld.t;
        }
        if (!wait_bounded(&ctl->empty[stage], phase ^ 1u, ctl, p, WAIT_SMEM_EMPTY, ld.t)) break;
        const int kx = ld.kb * C::kStageK;
        if (kPair) {
          // both CTAs' loads complete on the leader's barrier, which expects the bytes of both
          const uint32_t full_addr = map_to_cta(smem_u32(&ctl->full[stage]), 0);
          if (leader) mbar_arrive_expect_tx(&ctl->full[stage], C::kFullTxBytes);
#pragma unroll
          for (int at = 0; at < C::kAtoms; ++at) {
            tma_load_2d_pair_hint(smem_a + stage * C::kATileBytes + at * C::kAAtomBytes, &p.a_maps[ld.am], full_addr,
                                  kx + at * BK, ld.a_row, pol_a);
            uint8_t* b_dst = smem_b + stage * C::kBTileBytes + at * C::kBAtomBytes;
            if (p.b_mn_major) {
              // B is [K][N]: boxes of 64 columns (N) x 64 rows (K), one 8 KB chunk per 64 columns
#pragma unroll
              for (int ch = 0; ch < C::kBRows / 64; ++ch)
                tma_load_2d_pair_hint(b_dst + ch * kBChunkMnBytes, &p.b_maps[ld.bm], full_addr, ld.b_row + ch * 64, kx + at * BK, pol_b);
            } else {
              tma_load_2d_pair_hint(b_dst, &p.b_maps[ld.bm], full_addr, kx + at * BK, ld.b_row, pol_b);
            }
          }
        } else {
          mbar_arrive_expect_tx(&ctl->full[stage], C::kFullTxBytes);
#pragma unroll
          for (int at = 0; at < C::kAtoms; ++at) {
            tma_load_2d_hint(smem_a + stage * C::kATileBytes + at * C::kAAtomBytes, &p.a_maps[ld.am], &ctl->full[stage],
                             kx + at * BK, ld.a_row, pol_a);
            uint8_t* b_dst = smem_b + stage * C::kBTileBytes + at * C::kBAtomBytes;
            if (p.b_mn_major) {
#pragma unroll
              for (int ch = 0; ch < C::kBRows / 64; ++ch)
                tma_load_2d_hint(b_dst + ch * kBChunkMnBytes, &p.b_maps[ld.bm], &ctl->full[stage], ld.b_row + ch * 64, kx + at * BK, pol_b);
            } else {
              tma_load_2d_hint(b_dst, &p.b_maps[ld.bm], &ctl->full[stage], kx + at * BK, ld.b_row, pol_b);
            }
          }
        }
        if (p.prefetch_stages > 0 && !p.b_mn_major && pf.valid(p)) {
          const int px = pf.kb * C::kStageK;
#pragma unroll
          for (int at = 0; at < C::kAtoms; ++at) {
            tma_prefetch_l2_2d(&p.a_maps[pf.am], px + at * BK, pf.a_row);
            tma_prefetch_l2_2d(&p.b_maps[pf.bm], px + at * BK, pf.b_row);
          }
          pf.next(p);
        }
        ld.next(p);
        ++issued;
        if (++stage == C::kStages) {
          stage = 0;
          phase ^= 1u;
        }
      }
      // Do not leave the CTA while bulk copies may still be writing shared
      // memory: wait until the last fill of every stage has been consumed
      // (pair: the leader's barrier tracks both CTAs' copies) or has landed.
      const uint32_t outstanding = issued < uint32_t(C::kStages) ? issued : uint32_t(C::kStages);
      for (uint32_t i = 0; i < outstanding; ++i) {
        stage = (stage == 0) ? C::kStages - 1 : stage - 1;
        if (stage == C::kStages - 1) phase ^= 1u;
        if (kPair) {
          if (!wait_bounded(&ctl->empty[stage], phase, ctl, p, WAIT_DRAIN, -1)) break;
        } else {
          if (!wait_bounded(&ctl->full[stage], phase, ctl, p, WAIT_DRAIN, -1)) break;
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    // One lane runs the whole loop (a per-instruction "if (lane == 0)" inside a
    // 32-lane loop costs a divergence per MMA and slows the issue stream).
    if (leader && lane == 0) {
      const uint32_t idesc = umma_idesc_bf16_f32(kPair ? 2 * BM : BM, BN) | (p.b_mn_major ? kUmmaIdescBMnMajor : 0u);
      constexpr int kFullSteps = C::kStageK / UMMA_K;
      const uint64_t desc_a0 = umma_smem_desc_sw128(smem_u32(smem_a));
      const uint64_t desc_b0 = p.b_mn_major ? umma_smem_desc_sw128_mn(smem_u32(smem_b), kBChunkMnBytes)
                                            : umma_smem_desc_sw128(smem_u32(smem_b));
      // address-field step per 16-element k-step: 32 bytes inside a K-major swizzle row, two 8-row groups
      // (2048 bytes) in an N-contiguous chunk
      const uint32_t b_kstep = p.b_mn_major ? (2 * 1024) >> 4 : 2;
      int stage = 0;
      uint32_t phase = 0;
      uint32_t it = 0;
      bool ok = true;
      for (int t = unit; ok && t < p.total_tiles; t += n_units, ++it) {
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
          // descriptor address fields count 16-byte units
          const uint64_t da = desc_a0 + uint64_t((stage * C::kATileBytes) >> 4);
          const uint64_t db = desc_b0 + uint64_t((stage * C::kBTileBytes) >> 4);
          const uint32_t first = kb != 0 ? 1u : 0u;
          if (kb_in_seg != p.kb_per_seg - 1 || p.tail_ksteps == kFullSteps) {
#pragma unroll
            for (int ks = 0; ks < kFullSteps; ++ks) {
              // a 64-element atom holds 4 steps of 16 elements = 32 bytes each: +2 in the address field
              const uint64_t a_k = da + uint64_t(((ks >> 2) * C::kAAtomBytes >> 4) + (ks & 3) * 2);
              const uint64_t b_k = db + uint64_t(((ks >> 2) * C::kBAtomBytes >> 4) + (ks & 3) * b_kstep);
              if (kPair) umma_bf16_pair(d_tmem, a_k, b_k, idesc, ks ? 1u : first);
              else umma_bf16(d_tmem, a_k, b_k, idesc, ks ? 1u : first);
            }
          } else {
            for (int ks = 0; ks < p.tail_ksteps; ++ks) {
              const uint64_t a_k = da + uint64_t(((ks >> 2) * C::kAAtomBytes >> 4) + (ks & 3) * 2);
              const uint64_t b_k = db + uint64_t(((ks >> 2) * C::kBAtomBytes >> 4) + (ks & 3) * b_kstep);
              if (kPair) umma_bf16_pair(d_tmem, a_k, b_k, idesc, ks ? 1u : first);
              else umma_bf16(d_tmem, a_k, b_k, idesc, ks ? 1u : first);
            }
          }
          // the stage is reusable (in both CTAs) once these MMAs have read it
          if (kPair) umma_commit_pair(&ctl->empty[stage], 0x3);
          else umma_commit(&ctl->empty[stage]);
          if (++kb_in_seg == p.kb_per_seg) kb_in_seg = 0;
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (ok) {   // accumulator complete: wake the epilogue (of both CTAs)
          if (kPair) umma_commit_pair(&ctl->acc_full[buf], 0x3);
          else umma_commit(&ctl->acc_full[buf]);
        }
      }
      if (*reinterpret_cast<volatile int*>(&ctl->abort)) {
        // Gave up somewhere: wait for whatever the tensor core still has in
        // flight before tensor memory is released.
        if (kPair) umma_commit_pair(&ctl->drain, 0x1);
        else umma_commit(&ctl->drain);
        wait_bounded(&ctl->drain, 0, ctl, p, WAIT_DRAIN, -2);
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;               // TMEM lanes this warp may touch
    uint8_t* stage = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ctl + 1) + 15) & ~uintptr_t(15)) +
                     (warp - 2) * kStageWarpBytes;
    const int seg = lane & 7;                   // 16-byte segment of a 128-byte row piece this lane moves
    uint32_t it = 0;
    for (int t = unit; t < p.total_tiles; t += n_units, ++it) {
      const uint32_t buf = it & 1u;
      const uint32_t acc_phase = (it >> 1) & 1u;
      const TileCoord tc = decode_tile(p, t);
      const Frag frag = fragment_of(p, tc.blk, tc.mt * C::kTileRows + int(cta_rank) * BM);   // this CTA's 128 rows
      const BlockDesc& b = p.blocks[frag.blk];
      const int first_row = frag.r0 + quarter * 32;          // row (inside the block) of lane 0
      const int ncols = min(BN, p.N - tc.nt * BN);
      // SwiGLU halves the columns: accumulator columns (2j, 2j+1) = (gate, up) give output column j
      const int act = kAct ? p.activation : int(ACT_NONE);
      const int oshift = act == ACT_SWIGLU ? 1 : 0;
      const int ocols = ncols >> oshift;
      __nv_bfloat16* obase = p.out[b.out_idx] + int64_t(b.out_row0 + first_row) * p.ldo + ((int64_t(tc.nt) * BN) >> oshift);
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + buf * BN;
      const int npass = (ocols + 63) >> 6;

      if constexpr (kF32Sum) {
        // Ring read-modify-write with the running sum in FP32 scratch.  Same counters and ordering as below.  A
        // fragment's sum lies in the scratch in the order the lanes hold it (64 groups of 4 columns per warp, each
        // group the 32 lanes' 16 bytes in a row): a lane reads and writes its own row, every instruction of the
        // warp moves 512 contiguous bytes, and nothing passes through shared memory, whose bandwidth the tensor
        // core needs for its operands.  Four 32-column pieces are in flight ahead of the one being added.
        const bool live = frag.r0 < p.rows_per_block;          // a fragment past the block adds nothing
        const bool add_previous = live && b.step > 0;
        const bool last = int(b.step) == p.last_step;          // the owner's contribution: writes the BF16 result
        const int64_t frag_idx = (int64_t(b.part) * p.frags_m + frag.r0 / BM) * p.tiles_n + tc.nt;
        int* counter = p.tile_counters + frag_idx;
        uint4* sfrag = reinterpret_cast<uint4*>(p.ring_scratch + frag_idx * int64_t(BM * BN * 4)) + quarter * (BN / 4) * 32 + lane;
        const bool row_ok = first_row + lane < p.rows_per_block;
        uint4 ahead[4][8];
        auto fetch = [&](int piece, uint4 (&dst)[8]) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int g = piece * 8 + i;
            dst[i] = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok && g * 4 < ncols) dst[i] = __ldcg(sfrag + g * 32);       // written by another SM: from L2
          }
        };
        if (add_previous) {
          int ready = 1;
          if (lane == 0) ready = wait_counter(counter, int(b.step) * kEpilogueWarps, ctl, p, t) ? 1 : 0;
          ready = __shfl_sync(0xffffffffu, ready, 0);
          __syncwarp();      // orders the other lanes' loads behind lane 0's acquire
          if (!ready) break;
#pragma unroll
          for (int piece = 0; piece < 4; ++piece) fetch(piece, ahead[piece]);
        }
        if (!wait_bounded(&ctl->acc_full[buf], acc_phase, ctl, p, WAIT_ACC_FULL, t)) break;
        tc_fence_after_sync();
#pragma unroll
        for (int c = 0; c < BN / 32; ++c) {
          float prev[32];
          if (add_previous) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              prev[i * 4 + 0] = __uint_as_float(ahead[c & 3][i].x);
              prev[i * 4 + 1] = __uint_as_float(ahead[c & 3][i].y);
              prev[i * 4 + 2] = __uint_as_float(ahead[c & 3][i].z);
              prev[i * 4 + 3] = __uint_as_float(ahead[c & 3][i].w);
            }
            if (c + 4 < BN / 32) fetch(c + 4, ahead[c & 3]);
          }
          uint32_t v[32];
          tmem_ld_32x32b_x32(taddr + c * 32, v);
          tmem_ld_wait();
          if (c == BN / 32 - 1) {
            // accumulator fully copied to registers: hand it back to the MMA issuer
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
              if (kPair) mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->acc_empty[buf]), 0));
              else mbar_arrive(&ctl->acc_empty[buf]);
            }
          }
          if (add_previous) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + prev[i]);
          }
          if (c * 32 < ncols && live) {
            if (last) {
              // BF16 result: 64 bytes per row; every store instruction writes 8 rows x 64 contiguous bytes
              uint4* srow = reinterpret_cast<uint4*>(stage + lane * kStageRowBytes);
#pragma unroll
              for (int g = 0; g < 4; ++g)
                srow[g] = make_uint4(pack_bf16x2(__uint_as_float(v[g * 8 + 0]), __uint_as_float(v[g * 8 + 1])),
                                     pack_bf16x2(__uint_as_float(v[g * 8 + 2]), __uint_as_float(v[g * 8 + 3])),
                                     pack_bf16x2(__uint_as_float(v[g * 8 + 4]), __uint_as_float(v[g * 8 + 5])),
                                     pack_bf16x2(__uint_as_float(v[g * 8 + 6]), __uint_as_float(v[g * 8 + 7])));
              __syncwarp();
              const int col = c * 32 + (lane & 3) * 8;
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int r = i * 8 + (lane >> 2);
                if (first_row + r < p.rows_per_block && col < ncols)
                  *reinterpret_cast<uint4*>(obase + int64_t(r) * p.ldo + col) =
                      *reinterpret_cast<const uint4*>(stage + r * kStageRowBytes + (lane & 3) * 16);
              }
              __syncwarp();
            } else {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int g = c * 8 + i;
                if (row_ok && g * 4 < ncols) sfrag[g * 32] = make_uint4(v[i * 4 + 0], v[i * 4 + 1], v[i * 4 + 2], v[i * 4 + 3]);
              }
            }
          }
        }
        if (live) {
          // the warp barrier orders every lane's stores before lane 0's release of the counter
          __syncwarp();
          if (lane == 0) {
            int before;
            asm volatile("atom.add.release.gpu.global.s32 %0, [%1], 1;" : "=r"(before) : "l"(counter) : "memory");
            // the last warp of the last contributor leaves the counter at zero for the next call
            if (last && before == (p.last_step + 1) * kEpilogueWarps - 1) atomicExch(counter, 0);
          }
        }
        continue;
      }

      // Ring read-modify-write: contributor `step` of a partition adds its
      // partial tile to the running sum that contributor step-1 left in the
      // scratch, and passes the sum on there; the owner, last, writes it to its
      // rows instead.  One counter per 128 x 256 fragment of the output counts
      // the epilogue warps that have finished; contributor s starts when all
      // four warps of s-1 have.  (Per fragment, not per tile: the two CTAs of a
      // pair may be working on different partitions.)
      const bool rmw = p.epilogue == EPI_RING_RMW && frag.r0 < p.rows_per_block;   // a fragment past the block adds nothing
      const bool add_previous = rmw && b.step > 0;
      const bool pass_on = rmw && int(b.step) != p.last_step;    // not the owner's contribution: the sum goes to the scratch
      int* counter = nullptr;
      // The fragment's running sum lies in the scratch in the order the lanes hold it: 32 groups of 8 columns per
      // warp, each group the 32 lanes' 16 bytes in a row.  A lane reads and writes its own row, every instruction
      // of the warp moves 512 contiguous bytes, and nothing passes through shared memory, whose bandwidth the
      // tensor core needs for its operands.
      uint4* sfrag = nullptr;
      const bool row_ok = first_row + lane < p.rows_per_block;
      // `sum` first holds this lane's row of the running sum (packed BF16 pairs), then the row to store.
      uint32_t sum[BN / 2];
      if (rmw) {
        const int64_t frag_idx = (int64_t(b.part) * p.frags_m + frag.r0 / BM) * p.tiles_n + tc.nt;
        counter = p.tile_counters + frag_idx;
        sfrag = reinterpret_cast<uint4*>(p.ring_scratch + frag_idx * int64_t(BM * BN * 2)) + quarter * (BN / 8) * 32 + lane;
        if (add_previous) {
          // All of this happens while the tile's MMAs are still running: the wait for the previous
          // contributor and the fetch of its running sum need nothing from the accumulator.
          int ready = 1;
          if (lane == 0) ready = wait_counter(counter, int(b.step) * kEpilogueWarps, ctl, p, t) ? 1 : 0;
          ready = __shfl_sync(0xffffffffu, ready, 0);
          // lane 0 acquired the counter; the warp barrier orders the other lanes' loads of the running sum behind it
          __syncwarp();
          if (!ready) break;
          // all 32 loads of a lane in flight at once
#pragma unroll
          for (int g = 0; g < BN / 8; ++g) {
            uint4 piece = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok && g * 8 < ncols) piece = __ldcg(sfrag + g * 32);          // written by another SM: from L2
            sum[g * 4 + 0] = piece.x;
            sum[g * 4 + 1] = piece.y;
            sum[g * 4 + 2] = piece.z;
            sum[g * 4 + 3] = piece.w;
          }
        }
      }

      if (!wait_bounded(&ctl->acc_full[buf], acc_phase, ctl, p, WAIT_ACC_FULL, t)) break;
      tc_fence_after_sync();
      // 1) accumulator row (256 columns) TMEM -> registers 32 columns at a time, running sum added in FP32,
      //    packed to BF16 (sum[j] = output columns 2j, 2j+1)
#pragma unroll
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t v[32];
        tmem_ld_32x32b_x32(taddr + c * 32, v);
        tmem_ld_wait();
        if (add_previous) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint32_t o = sum[c * 16 + i];
            v[2 * i] = __float_as_uint(__uint_as_float(v[2 * i]) + __uint_as_float(o << 16));
            v[2 * i + 1] = __float_as_uint(__uint_as_float(v[2 * i + 1]) + __uint_as_float(o & 0xFFFF0000u));
          }
        }
        if (act == ACT_SWIGLU) {
          // 32 accumulator columns -> 16 output columns, packed densely from register 0 on
#pragma unroll
          for (int i = 0; i < 8; ++i)
            sum[c * 8 + i] = pack_bf16x2(swiglu_f32(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1])),
                                         swiglu_f32(__uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3])));
        } else {
          if (act == ACT_GELU_TANH) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(gelu_tanh_f32(__uint_as_float(v[i])));
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) sum[c * 16 + i] = pack_bf16x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
        }
      }
      // accumulator fully copied to registers: hand it back to the MMA issuer
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (kPair) mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->acc_empty[buf]), 0));
        else mbar_arrive(&ctl->acc_empty[buf]);
      }
      // 2) a contributor other than the owner passes the sum on through the scratch ...
      if (pass_on) {
#pragma unroll
        for (int g = 0; g < BN / 8; ++g)
          if (row_ok && g * 8 < ncols) sfrag[g * 32] = make_uint4(sum[g * 4 + 0], sum[g * 4 + 1], sum[g * 4 + 2], sum[g * 4 + 3]);
      }
      //    ... everything else goes registers -> padded shared memory -> global, 64 columns per pass: every store
      //    instruction writes 4 rows x 128 contiguous bytes.
#pragma unroll
      for (int pass = 0; pass < BN / 64; ++pass) {
        if (pass < npass && !pass_on) {
          uint4* srow = reinterpret_cast<uint4*>(stage + lane * kStageRowBytes);
#pragma unroll
          for (int g = 0; g < 8; ++g)
            srow[g] = make_uint4(sum[pass * 32 + g * 4 + 0], sum[pass * 32 + g * 4 + 1], sum[pass * 32 + g * 4 + 2],
                                 sum[pass * 32 + g * 4 + 3]);
          __syncwarp();
          const int col = pass * 64 + seg * 8;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = i * 4 + (lane >> 3);
            if (first_row + r < p.rows_per_block && col < ocols) {
              const uint4 q = *reinterpret_cast<const uint4*>(stage + r * kStageRowBytes + seg * 16);
              *reinterpret_cast<uint4*>(obase + int64_t(r) * p.ldo + col) = q;
            }
          }
          __syncwarp();
        }
      }
      if (rmw) {
        // The warp barrier orders every lane's stores before lane 0's release: the increment becomes visible
        // device-wide only after the rows this warp wrote (release is cumulative over what the barrier ordered).
        __syncwarp();
        if (lane == 0) {
          int before;
          asm volatile("atom.add.release.gpu.global.s32 %0, [%1], 1;" : "=r"(before) : "l"(counter) : "memory");
          // the last warp of the last contributor leaves the counter at zero for the next call
          if (int(b.step) == p.last_step && before == (p.last_step + 1) * kEpilogueWarps - 1) atomicExch(counter, 0);
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (kPair) {
    // the peer may still signal this CTA's barriers or read its shared memory
    cluster_arrive();
    cluster_wait();
  }
  if (warp == 1) {
    tc_fence_after_sync();
    if (kPair) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
  clock_record.end(p);
}

// ---- mixed-tile pair kernel ---------------------------------------------------------
//
// Same roles and protocol as gemm_kernel<true>, but a launch holds up to three kinds
// of tiles, all computed by a pair of CTAs:
//   big   512 x 256: each CTA owns 256 rows as two 128-row accumulators (TMEM
//         columns 0..255 and 256..511) that share one B tile.  A k-stage is one
//         64-wide atom: A block 0, A block 1, B = 3 chunks of 16 KB per CTA,
//         8 MMAs.  Per 128x256x64 MMA block the CTA loads 24 KB instead of 32.
//   small 256 x 256: one accumulator, k-stage = two 64-wide atoms (A0, A1, B0,
//         B1 = 4 chunks), 8 MMAs; accumulators alternate so the epilogue overlaps.
//   quarter 256 x 128: one 128-column accumulator, k-stage = two atoms of A and
//         this CTA's 64 B rows of both atoms in one chunk (3 chunks), 8 MMAs of
//         half the width; bound by operand delivery, used only where it lets
//         the last round over the pairs end sooner.
// Big tiles come first and fill whole waves (their number is a multiple of the
// number of pairs); the remaining slots are cut into small tiles and, last,
// quarter tiles, in the combination of whole rounds that ends soonest (the host
// decides).  Shared memory is one FIFO ring of 12 chunks; stage j uses barrier
// slot j & 3 with parity (j >> 2) & 1, and the producer fills stage j once stage
// j - depth has been released (depth 4 for big, 3 for small and quarter stages),
// which also holds across the changes of kind.
constexpr int kChunkBytes = BM * BK * 2;      // 16 KB: one 128-row, 64-column BF16 box
constexpr int kChunks = 12;
constexpr size_t kMixedSmemBytes =
    1024 + size_t(kChunks) * kChunkBytes + sizeof(Control) + 16 + size_t(kEpilogueWarps) * kStageWarpBytes;

struct MixedTile {
  int big;        // 1 = 512x256, 0 = 256x256 or 256x128
  int quarter;    // 1 = 256x128 (one 128-column half of a 256-column tile)
  int blk, nt;    // virtual block (p.group blocks), n-tile (256 columns)
  int col0;       // first output column of the tile
  int row0;       // first row of the pair's tile inside the virtual block
  int valid;
};
__device__ __forceinline__ MixedTile decode_mixed(const GemmParams& p, int t) {
  MixedTile m;
  int tb;
  int half = 0, nq = 0;
  m.quarter = 0;
  if (t < p.n_big) {
    m.big = 1;
    tb = t;
  } else if (p.h_last == 2) {
    m.big = 0;
    if (t < p.n_small_end) {
      const int u = t - p.n_big;
      tb = p.n_big + (u >> 1);
      half = u & 1;
    } else {
      // the last slots of the launch as four 256x128 tiles each: the remainder then fills the pairs more evenly
      const int u = t - p.n_small_end;
      tb = p.n_big + ((p.n_small_end - p.n_big) >> 1) + (u >> 2);
      half = (u >> 1) & 1;
      nq = u & 1;
      m.quarter = 1;
    }
  } else {
    // A block's last 512-row slot holds at most 256 rows (then the launch has no 512x256 tiles): its second
    // half does not exist and is not numbered, so that every tile index is a tile and consecutive indices
    // spread evenly over the pairs.  Per block: full slot rows (2 halves x tiles_n), then the short one.
    m.big = 0;
    const int per_block_small = (2 * (p.big_tiles_m - 1) + 1) * p.tiles_n;
    m.blk = t / per_block_small;
    int w = t - m.blk * per_block_small;
    const int full = 2 * (p.big_tiles_m - 1) * p.tiles_n;
    int mtb;
    if (w < full) {
      mtb = w / (2 * p.tiles_n);
      w -= mtb * 2 * p.tiles_n;
      m.nt = w >> 1;
      half = w & 1;
    } else {
      mtb = p.big_tiles_m - 1;
      m.nt = w - full;
    }
    m.row0 = mtb * (4 * BM) + half * (2 * BM);
    m.col0 = m.nt * BN;
    m.valid = m.row0 < p.vrows;
    return m;
  }
  const int per_block = p.big_tiles_m * p.tiles_n;
  m.blk = tb / per_block;
  const int w = tb - m.blk * per_block;
  const int mtb = w / p.tiles_n;
  m.nt = w - mtb * p.tiles_n;
  m.row0 = mtb * (4 * BM) + half * (2 * BM);
  m.col0 = m.nt * BN + nq * (BN / 2);
  m.valid = m.row0 < p.vrows && m.col0 < p.N;      // the second half of a ragged last column tile may not exist
  return m;
}

// Walks the k-stages of one pair's tiles: tile, K segment, k-stage.
struct MixedIter {
  int t, step, cta_rank;
  int seg, kb, n_kb;
  MixedTile tile;
  int blk0, blk1;            // blocks of this CTA's 128-row fragments (blk1: second fragment of a 512x256 tile)
  int am, am1, bm, a_row, a_row1, b_row;
  __device__ MixedIter(const GemmParams& p, int unit, int n_units, int rank) : t(unit), step(n_units), cta_rank(rank), seg(0), kb(0) {
    skip_invalid(p);
  }
  __device__ bool valid(const GemmParams& p) const { return t < p.total_tiles; }
  __device__ void skip_invalid(const GemmParams& p) {
    while (t < p.total_tiles) {
      tile = decode_mixed(p, t);
      if (tile.valid) {
        enter(p);
        return;
      }
      t += step;
    }
  }
  __device__ void enter(const GemmParams& p) {
    const int v0 = tile.row0 + cta_rank * (tile.big ? 2 * BM : BM);
    const Frag f0 = fragment_of(p, tile.blk, v0);
    const Frag f1 = tile.big ? fragment_of(p, tile.blk, v0 + BM) : f0;
    const BlockDesc& b0 = p.blocks[f0.blk];
    const BlockDesc& b1 = p.blocks[f1.blk];
    blk0 = f0.blk;
    blk1 = f1.blk;
    a_row = b0.a_row0 + f0.r0;
    a_row1 = b1.a_row0 + f1.r0;
    b_row = tile.col0 + cta_rank * (tile.quarter ? BN / 4 : BN / 2);  // this CTA's half of the tile's B rows
    am = (p.n_seg > 1) ? p.seg_rank[tile.blk][seg] : b0.a_map;      // segmented K: blocks are never grouped
    am1 = (p.n_seg > 1) ? am : b1.a_map;
    bm = (p.n_seg > 1) ? am : b0.b_map;                             // the blocks of a group share their B tensor
    n_kb = tile.big ? p.kb_big : p.kb_per_seg;
  }
  __device__ void next(const GemmParams& p) {
    if (++kb < n_kb) return;
    kb = 0;
    if (++seg == p.n_seg) {
      seg = 0;
      t += step;
      skip_invalid(p);
      return;
    }
    enter(p);
  }
};

// kAct: the epilogue applies p.activation.  A separate instantiation, because the extra code in the
// accumulator-read phase (which the MMA issuer waits for) slows the plain store down by 1-3 %.
template <bool kAct>
__global__ void __launch_bounds__(kThreads, 1) gemm_mixed_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
  Control* ctl = reinterpret_cast<Control*>(smem + kChunks * kChunkBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = cluster_ctarank();
  const bool leader = cta_rank == 0;
  const int unit = int(blockIdx.x >> 1);
  const int n_units = int(gridDim.x >> 1);
  ClockRecord clock_record;
  clock_record.begin();

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->acc_full[b], 1);
      mbar_init(&ctl->acc_empty[b], 2 * kEpilogueWarps);
    }
    mbar_init(&ctl->drain, 1);
    ctl->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(&ctl->tmem_base, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const uint64_t pol_a = make_l2_policy(p.a_hint);
      const uint64_t pol_b = make_l2_policy(p.b_hint);
      uint32_t j = 0;          // global stage counter
      int chunk = 0;           // ring cursor
      int ready_t = -1;
      for (MixedIter it(p, unit, n_units, int(cta_rank)); it.valid(p); it.next(p), ++j) {
        if (it.t != ready_t) {      // first stage of a tile: its A rows may still be on their way
          if (!wait_ready_flag(p, p.blocks[it.blk0], ctl, it.t)) break;
          if (it.blk1 != it.blk0 && !wait_ready_flag(p, p.blocks[it.blk1], ctl, it.t)) break;
          ready_t = it.t;
        }
        const int big = it.tile.big;
        // A 512x256 stage (3 chunks) follows only stages of its own kind: four of them fill the ring.  A 256x256
        // stage (4 chunks) or a 256x128 stage (3 chunks, possibly behind 4-chunk stages) overwrites nothing newer
        // than the third stage before it.
        const uint32_t depth = big ? 4u : 3u;
        if (j >= depth) {
          const uint32_t r = j - depth;      // this stage's chunks are free once stage r has been released
          if (!wait_bounded(&ctl->empty[r & 3u], (r >> 2) & 1u, ctl, p, WAIT_SMEM_EMPTY, it.t)) break;
        }
        const uint32_t slot = j & 3u;
        const uint32_t full_addr = map_to_cta(smem_u32(&ctl->full[slot]), 0);
        const int quarter = it.tile.quarter;
        const int nchunks = (big || quarter) ? 3 : 4;
        if (leader) mbar_arrive_expect_tx(&ctl->full[slot], uint32_t(2 * nchunks * kChunkBytes));
        uint8_t* c0 = smem + ((chunk + 0) % kChunks) * kChunkBytes;
        uint8_t* c1 = smem + ((chunk + 1) % kChunks) * kChunkBytes;
        uint8_t* c2 = smem + ((chunk + 2) % kChunks) * kChunkBytes;
        // this CTA's 128 rows of B for one 64-wide k-atom: one box when B is [N][K], two boxes of 64 columns
        // (8 KB chunks) when B is [K][N]
        auto load_b = [&](uint8_t* dst, int kx) {
          if (p.b_mn_major) {
            tma_load_2d_pair_hint(dst, &p.b_maps[it.bm], full_addr, it.b_row, kx, pol_b);
            tma_load_2d_pair_hint(dst + kBChunkMnBytes, &p.b_maps[it.bm], full_addr, it.b_row + 64, kx, pol_b);
          } else {
            tma_load_2d_pair_hint(dst, &p.b_maps[it.bm], full_addr, kx, it.b_row, pol_b);
          }
        };
        if (big) {
          const int kx = it.kb * BK;
          tma_load_2d_pair_hint(c0, &p.a_maps[it.am], full_addr, kx, it.a_row, pol_a);
          tma_load_2d_pair_hint(c1, &p.a_maps[it.am1], full_addr, kx, it.a_row1, pol_a);
          load_b(c2, kx);
        } else if (quarter) {
          // 256x128 tile: two k-atoms of A (chunks 0, 1) and this CTA's 64 B rows of both atoms in the two halves
          // of chunk 2 (8 KB boxes: 64 rows x 64 columns from the 64-row-box maps, or one 64x64 box of a [K][N] weight)
          const int kx = it.kb * 2 * BK;
          tma_load_2d_pair_hint(c0, &p.a_maps[it.am], full_addr, kx, it.a_row, pol_a);
          tma_load_2d_pair_hint(c1, &p.a_maps[it.am], full_addr, kx + BK, it.a_row, pol_a);
          if (p.b_mn_major) {
            tma_load_2d_pair_hint(c2, &p.b_maps[it.bm], full_addr, it.b_row, kx, pol_b);
            tma_load_2d_pair_hint(c2 + kBChunkMnBytes, &p.b_maps[it.bm], full_addr, it.b_row, kx + BK, pol_b);
          } else {
            tma_load_2d_pair_hint(c2, &p.b_maps_q[it.bm], full_addr, kx, it.b_row, pol_b);
            tma_load_2d_pair_hint(c2 + kChunkBytes / 2, &p.b_maps_q[it.bm], full_addr, kx + BK, it.b_row, pol_b);
          }
        } else {
          const int kx = it.kb * 2 * BK;
          uint8_t* c3 = smem + ((chunk + 3) % kChunks) * kChunkBytes;
          tma_load_2d_pair_hint(c0, &p.a_maps[it.am], full_addr, kx, it.a_row, pol_a);
          load_b(c2, kx);
          tma_load_2d_pair_hint(c1, &p.a_maps[it.am], full_addr, kx + BK, it.a_row, pol_a);
          load_b(c3, kx + BK);
        }
        chunk = (chunk + nchunks) % kChunks;
      }
      // wait until the last stages have been consumed (the leader's MMAs read both CTAs' chunks)
      const uint32_t back = j < 4u ? j : 4u;
      for (uint32_t i = 1; i <= back; ++i) {
        const uint32_t r = j - i;
        if (!wait_bounded(&ctl->empty[r & 3u], (r >> 2) & 1u, ctl, p, WAIT_DRAIN, -1)) break;
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    // One lane runs the whole loop: a per-instruction "if (lane == 0)" inside a
    // 32-lane loop costs a divergence per MMA and measurably slows the issue stream.
    if (leader && lane == 0) {
      const uint32_t idesc = umma_idesc_bf16_f32(2 * BM, BN) | (p.b_mn_major ? kUmmaIdescBMnMajor : 0u);
      const uint32_t idesc_q = umma_idesc_bf16_f32(2 * BM, BN / 2) | (p.b_mn_major ? kUmmaIdescBMnMajor : 0u);
      const uint64_t desc0 = umma_smem_desc_sw128(smem_u32(smem));
      // B chunks: the same ring, but an N-contiguous chunk is two 8 KB sub-chunks and a k-step is 2048 bytes
      const uint64_t desc0b = p.b_mn_major ? umma_smem_desc_sw128_mn(smem_u32(smem), kBChunkMnBytes) : desc0;
      const uint32_t bk = p.b_mn_major ? (2 * 1024) >> 4 : 2;
      uint32_t j = 0;
      int chunk = 0;
      uint32_t uses0 = 0, uses1 = 0;      // completed uses of accumulator 0 / 1
      uint32_t small_rr = 0;
      bool ok = true;
      for (int t = unit; ok && t < p.total_tiles; t += n_units) {
        const MixedTile tile = decode_mixed(p, t);
        if (!tile.valid) continue;
        const int big = tile.big;
        const int kb_seg = big ? p.kb_big : p.kb_per_seg;
        const int n_kb = kb_seg * p.n_seg;
        const int tail = big ? p.tail_big : p.tail_ksteps;
        const uint32_t buf = big ? 0u : (small_rr & 1u);
        // the accumulator(s) this tile writes must have been drained by the epilogue
        if (!wait_bounded(&ctl->acc_empty[buf], ((buf ? uses1 : uses0) & 1u) ^ 1u, ctl, p, WAIT_ACC_EMPTY, t)) break;
        tc_fence_after_sync();
        if (big) {
          // 512x256 tile: A block 0 -> accumulator 0, A block 1 -> accumulator 1, both with the stage's B chunk.
          // In the body of the tile the two MMAs of a k-step are adjacent so that they read the same B slice
          // back to back.  Both accumulators are live for the whole tile, so nothing hides the epilogue
          // unless the two are skewed at the tile's ends: for the first and the last `skew` stages all of
          // accumulator 0's MMAs are issued before accumulator 1's.  Accumulator 0 is then complete `skew`
          // half-stages before the tile ends (the epilogue reads it while accumulator 1 finishes) and the
          // next tile starts on it while the epilogue still drains accumulator 1.
          const int skew = (n_kb >= 2 * p.skew) ? p.skew : 0;
          auto ksteps = [&](int kb) { return (kb % kb_seg == kb_seg - 1) ? tail : BK / UMMA_K; };
          auto issue = [&](uint32_t acc, int a_chunk, int b_chunk, int nk, uint32_t first) {
            const uint64_t da = desc0 + uint64_t(((a_chunk % kChunks) * kChunkBytes) >> 4);
            const uint64_t db = desc0b + uint64_t(((b_chunk % kChunks) * kChunkBytes) >> 4);
            if (nk == BK / UMMA_K) {
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k) umma_bf16_pair(acc, da + uint64_t(k * 2), db + uint64_t(k * bk), idesc, k ? 1u : first);
            } else {
              for (int k = 0; k < nk; ++k) umma_bf16_pair(acc, da + uint64_t(k * 2), db + uint64_t(k * bk), idesc, k ? 1u : first);
            }
          };
          // `count` stages from stage kb on, accumulator 0 first, then accumulator 1 (which releases the stages)
          auto skewed = [&](int kb, int count, bool wait_acc1) -> bool {
            for (int s = 0; s < count; ++s) {
              if (!wait_bounded(&ctl->full[(j + s) & 3u], ((j + s) >> 2) & 1u, ctl, p, WAIT_SMEM_FULL, t)) return false;
              tc_fence_after_sync();
              issue(tmem_base, chunk + 3 * s, chunk + 3 * s + 2, ksteps(kb + s), (kb + s) != 0 ? 1u : 0u);
            }
            if (wait_acc1) {
              if (!wait_bounded(&ctl->acc_empty[1], (uses1 & 1u) ^ 1u, ctl, p, WAIT_ACC_EMPTY, t)) return false;
              tc_fence_after_sync();
            } else {
              umma_commit_pair(&ctl->acc_full[0], 0x3);
            }
            for (int s = 0; s < count; ++s) {
              issue(tmem_base + BN, chunk + 3 * s + 1, chunk + 3 * s + 2, ksteps(kb + s), (kb + s) != 0 ? 1u : 0u);
              umma_commit_pair(&ctl->empty[(j + s) & 3u], 0x3);
            }
            j += uint32_t(count);
            chunk = (chunk + 3 * count) % kChunks;
            return true;
          };
          int kb = 0;
          if (skew) {
            if (!skewed(0, skew, true)) { ok = false; break; }
            kb = skew;
          } else {
            if (!wait_bounded(&ctl->acc_empty[1], (uses1 & 1u) ^ 1u, ctl, p, WAIT_ACC_EMPTY, t)) break;
            tc_fence_after_sync();
          }
          for (; kb < n_kb - skew; ++kb, ++j) {
            if (!wait_bounded(&ctl->full[j & 3u], (j >> 2) & 1u, ctl, p, WAIT_SMEM_FULL, t)) {
              ok = false;
              break;
            }
            tc_fence_after_sync();
            const uint64_t d0 = desc0 + uint64_t((((chunk + 0) % kChunks) * kChunkBytes) >> 4);
            const uint64_t d1 = desc0 + uint64_t((((chunk + 1) % kChunks) * kChunkBytes) >> 4);
            const uint64_t d2 = desc0b + uint64_t((((chunk + 2) % kChunks) * kChunkBytes) >> 4);
            const uint32_t first = kb != 0 ? 1u : 0u;
            const int nk = ksteps(kb);
            if (nk == BK / UMMA_K) {
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k) {
                umma_bf16_pair(tmem_base, d0 + uint64_t(k * 2), d2 + uint64_t(k * bk), idesc, k ? 1u : first);
                umma_bf16_pair(tmem_base + BN, d1 + uint64_t(k * 2), d2 + uint64_t(k * bk), idesc, k ? 1u : first);
              }
            } else {
              for (int k = 0; k < nk; ++k) {
                umma_bf16_pair(tmem_base, d0 + uint64_t(k * 2), d2 + uint64_t(k * bk), idesc, k ? 1u : first);
                umma_bf16_pair(tmem_base + BN, d1 + uint64_t(k * 2), d2 + uint64_t(k * bk), idesc, k ? 1u : first);
              }
            }
            chunk = (chunk + 3) % kChunks;
            umma_commit_pair(&ctl->empty[j & 3u], 0x3);      // the stage is reusable in both CTAs once these MMAs have read it
          }
          if (!ok) break;
          if (skew) {
            if (!skewed(n_kb - skew, skew, false)) { ok = false; break; }
          } else {
            umma_commit_pair(&ctl->acc_full[0], 0x3);
          }
          umma_commit_pair(&ctl->acc_full[1], 0x3);
          ++uses0;
          ++uses1;
        } else {
          // 256x256: A atoms in chunks 0 and 1, B atoms in chunks 2 and 3.  256x128: the two B atoms (64 rows per CTA)
          // share chunk 2, and the MMA is 128 columns wide.
          const int quarter = tile.quarter;
          const uint32_t idesc_t = quarter ? idesc_q : idesc;
          const uint32_t acc_a = tmem_base + buf * BN;
          int kb_in_seg = 0;
          for (int kb = 0; kb < n_kb; ++kb, ++j) {
            if (!wait_bounded(&ctl->full[j & 3u], (j >> 2) & 1u, ctl, p, WAIT_SMEM_FULL, t)) {
              ok = false;
              break;
            }
            tc_fence_after_sync();
            const bool full_stage = kb_in_seg != kb_seg - 1 || tail == 2 * BK / UMMA_K;
            const uint64_t d0 = desc0 + uint64_t((((chunk + 0) % kChunks) * kChunkBytes) >> 4);
            const uint64_t d1 = desc0 + uint64_t((((chunk + 1) % kChunks) * kChunkBytes) >> 4);
            const uint64_t d2 = desc0b + uint64_t((((chunk + 2) % kChunks) * kChunkBytes) >> 4);
            const uint64_t d3 = quarter ? d2 + uint64_t((kChunkBytes / 2) >> 4)
                                        : desc0b + uint64_t((((chunk + 3) % kChunks) * kChunkBytes) >> 4);
            const uint32_t first = kb != 0 ? 1u : 0u;
            if (full_stage) {
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k) umma_bf16_pair(acc_a, d0 + uint64_t(k * 2), d2 + uint64_t(k * bk), idesc_t, k ? 1u : first);
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k) umma_bf16_pair(acc_a, d1 + uint64_t(k * 2), d3 + uint64_t(k * bk), idesc_t, 1u);
            } else {
              for (int ks = 0; ks < tail; ++ks) {
                const int k = ks & 3;
                umma_bf16_pair(acc_a, ((ks >> 2) ? d1 : d0) + uint64_t(k * 2), ((ks >> 2) ? d3 : d2) + uint64_t(k * bk), idesc_t,
                               ks ? 1u : first);
              }
            }
            chunk = (chunk + (quarter ? 3 : 4)) % kChunks;
            umma_commit_pair(&ctl->empty[j & 3u], 0x3);
            if (++kb_in_seg == kb_seg) kb_in_seg = 0;
          }
          if (!ok) break;
          umma_commit_pair(&ctl->acc_full[buf], 0x3);
          if (buf) ++uses1; else ++uses0;
          ++small_rr;
        }
      }
      if (*reinterpret_cast<volatile int*>(&ctl->abort)) {
        // gave up somewhere: let the tensor core finish what it still has before tensor memory is released
        umma_commit_pair(&ctl->drain, 0x1);
        wait_bounded(&ctl->drain, 0, ctl, p, WAIT_DRAIN, -2);
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;
    uint8_t* stage = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ctl + 1) + 15) & ~uintptr_t(15)) +
                     (warp - 2) * kStageWarpBytes;
    uint32_t uses0 = 0, uses1 = 0, small_rr = 0;
    bool ok = true;
    for (int t = unit; ok && t < p.total_tiles; t += n_units) {
      const MixedTile tile = decode_mixed(p, t);
      if (!tile.valid) continue;
      const int ncols = min(tile.quarter ? BN / 2 : BN, p.N - tile.col0);
      const int n_acc = tile.big ? 2 : 1;
      for (int a = 0; a < n_acc && ok; ++a) {
        const uint32_t buf = tile.big ? uint32_t(a) : (small_rr & 1u);
        const uint32_t n = buf ? uses1 : uses0;
        if (!wait_bounded(&ctl->acc_full[buf], n & 1u, ctl, p, WAIT_ACC_FULL, t)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        // big: this CTA owns rows [256*rank, +256) of the tile, accumulator a holds its 128-row fragment a
        const Frag frag = fragment_of(p, tile.blk, tile.row0 + (tile.big ? int(cta_rank) * 2 * BM + a * BM : int(cta_rank) * BM));
        const BlockDesc& b = p.blocks[frag.blk];
        const int row_in_block = frag.r0 + quarter * 32 + lane;
        // SwiGLU halves the columns: accumulator columns (2j, 2j+1) = (gate, up) give output column j
        const int act = kAct ? p.activation : int(ACT_NONE);
        const int oshift = act == ACT_SWIGLU ? 1 : 0;
        const int ocols = ncols >> oshift;
        __nv_bfloat16* orow = p.out[b.out_idx] + int64_t(b.out_row0 + row_in_block) * p.ldo + (int64_t(tile.col0) >> oshift);
        const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + buf * BN;
        const int first_row = row_in_block - lane;          // row of lane 0
        __nv_bfloat16* obase = orow - int64_t(lane) * p.ldo;
        // 1) The whole accumulator row (256 columns) goes TMEM -> registers as packed BF16, then the
        //    accumulator is handed back at once: with two live accumulators per tile the MMA issuer
        //    waits for this, so the time TMEM is held matters more than the time the stores take.
        //    (A 256x128 tile uses the first 128 columns; the rest is read too and never stored.)
        uint32_t packed[BN / 2];
#pragma unroll
        for (int c = 0; c < BN / 64; ++c) {
          uint32_t v[32], w[32];
          tmem_ld_32x32b_x32(taddr + c * 64, v);
          tmem_ld_32x32b_x32(taddr + c * 64 + 32, w);
          tmem_ld_wait();
          if (act == ACT_SWIGLU) {
            // 64 accumulator columns -> 32 output columns, packed densely from register 0 on
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              packed[c * 16 + i] = pack_bf16x2(swiglu_f32(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1])),
                                               swiglu_f32(__uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3])));
              packed[c * 16 + 8 + i] = pack_bf16x2(swiglu_f32(__uint_as_float(w[4 * i]), __uint_as_float(w[4 * i + 1])),
                                                   swiglu_f32(__uint_as_float(w[4 * i + 2]), __uint_as_float(w[4 * i + 3])));
            }
          } else {
            if (act == ACT_GELU_TANH) {
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                v[i] = __float_as_uint(gelu_tanh_f32(__uint_as_float(v[i])));
                w[i] = __float_as_uint(gelu_tanh_f32(__uint_as_float(w[i])));
              }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              packed[c * 32 + i] = pack_bf16x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
              packed[c * 32 + 16 + i] = pack_bf16x2(__uint_as_float(w[2 * i]), __uint_as_float(w[2 * i + 1]));
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->acc_empty[buf]), 0));
        // 2) registers -> padded shared memory -> global, 64 columns per pass: every store
        //    instruction writes 4 rows x 128 contiguous bytes.
        const int npass = (ocols + 63) >> 6;
        const int seg = lane & 7;
#pragma unroll
        for (int pass = 0; pass < BN / 64; ++pass) {
          if (pass < npass) {
            uint4* srow = reinterpret_cast<uint4*>(stage + lane * kStageRowBytes);
#pragma unroll
            for (int g = 0; g < 8; ++g)
              srow[g] = make_uint4(packed[pass * 32 + g * 4 + 0], packed[pass * 32 + g * 4 + 1], packed[pass * 32 + g * 4 + 2],
                                   packed[pass * 32 + g * 4 + 3]);
            __syncwarp();
            const int col = pass * 64 + seg * 8;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = i * 4 + (lane >> 3);
              if (first_row + r < p.rows_per_block && col < ocols) {
                const uint4 q = *reinterpret_cast<const uint4*>(stage + r * kStageRowBytes + seg * 16);
                *reinterpret_cast<uint4*>(obase + int64_t(r) * p.ldo + col) = q;
              }
            }
            __syncwarp();
          }
        }
        if (buf) ++uses1; else ++uses0;
      }
      if (!tile.big) ++small_rr;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
  clock_record.end(p);
}

// ---- host side ----------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  // looked up once; the initialisation of a function-local static is thread-safe
  static const EncodeTiledFn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(ptr);
    return static_cast<EncodeTiledFn>(nullptr);
  }();
  return fn;
}

// K-major BF16 matrix [rows x K]; box = BK columns x box_rows rows, 128-byte swizzle, zero fill outside.
bool encode_kmajor_uncached(CUtensorMap* map, const void* ptr, int64_t rows, int64_t K, int box_rows) {
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

// Encoded tensor maps are kept per host thread in a small 4-way set-associative table keyed by everything the
// encoding depends on (base pointer, rows, row length, box rows): a training loop calls the same operator
// on the same buffers over and over, and the driver call costs about a microsecond per map (2P maps per
// fused launch, d times that for InterDecom).  A map describes addresses and shapes, not contents, so an
// entry never goes stale; a different pointer or shape is a different key and is encoded afresh.
struct MapCache {
  static constexpr int kSets = 64, kWays = 4;
  struct Key {
    const void* ptr;
    int64_t rows, cols;
    int32_t box_rows, valid;
  };
  Key key[kSets][kWays] = {};
  uint8_t next_way[kSets] = {};          // round-robin replacement inside a set
  alignas(64) CUtensorMap map[kSets][kWays];
};
std::atomic<uint64_t> g_map_hits{0}, g_map_misses{0};

bool encode_kmajor(CUtensorMap* map, const void* ptr, int64_t rows, int64_t K, int box_rows) {
  static thread_local MapCache cache;
  uint64_t h = uint64_t(reinterpret_cast<uintptr_t>(ptr)) >> 4;
  h = (h ^ (h >> 17) ^ (uint64_t(rows) * 0x9E3779B97F4A7C15ull) ^ (uint64_t(K) * 0xC2B2AE3D27D4EB4Full) ^ uint64_t(box_rows)) *
      0xD6E8FEB86659FD93ull;
  const int set = int(h >> 58) & (MapCache::kSets - 1);
  for (int w = 0; w < MapCache::kWays; ++w) {
    const MapCache::Key& k = cache.key[set][w];
    if (k.valid && k.ptr == ptr && k.rows == rows && k.cols == K && k.box_rows == box_rows) {
      *map = cache.map[set][w];
      g_map_hits.fetch_add(1, std::memory_order_relaxed);
      return true;
    }
  }
  int way = -1;
  for (int w = 0; w < MapCache::kWays && way < 0; ++w)
    if (!cache.key[set][w].valid) way = w;
  if (way < 0) {
    way = cache.next_way[set];
    cache.next_way[set] = uint8_t((way + 1) % MapCache::kWays);
  }
  MapCache::Key& k = cache.key[set][way];
  if (!encode_kmajor_uncached(&cache.map[set][way], ptr, rows, K, box_rows)) {
    k.valid = 0;
    return false;
  }
  k.ptr = ptr;
  k.rows = rows;
  k.cols = K;
  k.box_rows = box_rows;
  k.valid = 1;
  *map = cache.map[set][way];
  g_map_misses.fetch_add(1, std::memory_order_relaxed);
  return true;
}

struct DeviceInfo {
  int num_sms = 0;
  int max_pairs = 0;     // co-resident clusters of two CTAs of the pair kernel
  bool ready = false;
};

// Per-device facts, gathered the first time a device launches (function attributes and cluster
// occupancy belong to the device that is current).
int device_info(DeviceInfo** out) {
  constexpr int kMaxDevices = 64;
  static DeviceInfo infos[kMaxDevices];
  static std::mutex mu;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevices) return COMPASS_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  DeviceInfo& info = infos[dev];
  if (!info.ready) {
    e = cudaDeviceGetAttribute(&info.num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_kernel<false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_bytes<false>()));
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_kernel<false, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_bytes<false>()));
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_bytes<false>()));
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_kernel<true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_bytes<true>()));
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_kernel<true, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_bytes<true>()));
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem_bytes<true>()));
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_mixed_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kMixedSmemBytes));
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(gemm_mixed_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kMixedSmemBytes));
    if (e != cudaSuccess) return record_cuda_error(e);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(info.num_sms / 2 * 2));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes<true>();
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, gemm_kernel<true, false, false>, &cfg);
    if (e != cudaSuccess) return record_cuda_error(e);
    info.max_pairs = clusters;
    info.ready = true;
  }
  *out = &info;
  return COMPASS_OK;
}

}  // namespace

void tensor_map_cache_stats(uint64_t* hits, uint64_t* misses) {
  *hits = g_map_hits.load(std::memory_order_relaxed);
  *misses = g_map_misses.load(std::memory_order_relaxed);
}

size_t gemm_smem_bytes() {
  size_t m = smem_bytes<true>() > smem_bytes<false>() ? smem_bytes<true>() : smem_bytes<false>();
  return m > kMixedSmemBytes ? m : kMixedSmemBytes;
}

int gemm_tile_rows(int mode, int rows_per_block) {
  const bool pair = mode == GEMM_MODE_PAIR || (mode == GEMM_MODE_AUTO && rows_per_block >= 2 * BM);
  return pair ? 2 * BM : BM;
}

// How the blocks of a launch are tiled (pure host arithmetic; see TilePlan in internal.h).
TilePlan plan_tiles(const GemmLaunch& L, int max_pairs) {
  TilePlan t = {};
  t.sub_pad = (L.rows_per_block + BM - 1) / BM * BM;
  t.group = 1;
  if (L.mode == GEMM_MODE_SINGLE || max_pairs <= 0) {
    t.pair = 0;
  } else if (L.mode == GEMM_MODE_PAIR || t.sub_pad >= 2 * BM) {
    t.pair = 1;
  } else {
    // One 128-row fragment per block: a CTA pair takes fragments of `group` consecutive blocks that read the
    // same B tensor (for the fused operators: the two ring entries of one step of a rank, adjacent in that
    // rank's schedule order).  Segmented K cannot group: its blocks walk the B tensors in different orders.
    t.pair = 0;
    if (L.n_seg == 1 && L.share_run >= 2 && L.n_blocks % L.share_run == 0) {
      for (int g = 2; g <= L.share_run; ++g)
        if (L.share_run % g == 0) {
          t.group = g;
          t.pair = 1;
          break;
        }
    }
  }
  const int tile_rows = t.pair ? 2 * BM : BM;
  t.vrows = t.group * t.sub_pad;
  t.n_vblocks = L.n_blocks / t.group;
  t.tiles_m = (t.vrows + tile_rows - 1) / tile_rows;
  t.tiles_n = int((L.N + BN - 1) / BN);
  t.total_tiles = t.n_vblocks * t.tiles_m * t.tiles_n;
  t.n_small = t.total_tiles;
  // Mixed tiles: 512x256 for as many whole waves of pairs as the launch holds, smaller ones for the rest.
  t.mixed = t.pair && L.epilogue == EPI_STORE && L.mode != GEMM_MODE_PAIR;
  if (!t.mixed || t.total_tiles <= 0) return t;
  // rows of a (virtual) block that hold data when it is cut into 256-row halves of 512-row slots
  const int rows = t.group > 1 ? t.vrows : L.rows_per_block;
  t.vrows = rows;
  t.big_tiles_m = (rows + 4 * BM - 1) / (4 * BM);
  const int total_big = t.n_vblocks * t.big_tiles_m * t.tiles_n;
  const bool use_big = rows % (4 * BM) == 0;
  t.n_big = use_big ? (total_big / max_pairs) * max_pairs : 0;
  t.h_last = (rows - (t.big_tiles_m - 1) * 4 * BM > 2 * BM) ? 2 : 1;
  if (t.h_last == 2) {
    // The slots left after the whole waves of 512x256 tiles are cut into 256x256 tiles (two per slot, half a big
    // tile's time each) and, last, 256x128 tiles (four per slot; their stages carry 48 KB of operands for half the
    // MMA work, so they are bound by operand delivery: measured 0.42 of a big tile's time each), in the combination
    // of whole rounds over the pairs that ends soonest.
    const int remaining = total_big - t.n_big;
    int small_slots = remaining;
    if (t.n_big > 0 && remaining > 0) {
      double best = 1e30;
      for (int r1 = (2 * remaining + max_pairs - 1) / max_pairs; r1 >= 0; --r1) {
        const int s_slots = std::min(remaining, (r1 * max_pairs) / 2);
        const int r2 = (4 * (remaining - s_slots) + max_pairs - 1) / max_pairs;
        const double cost = 0.5 * r1 + 0.42 * r2;
        if (cost < best - 1e-9) {
          best = cost;
          small_slots = s_slots;
        }
      }
    }
    t.n_small = 2 * small_slots;
    t.n_quarter = 4 * (remaining - small_slots);
  } else {
    // a block's last 512-row slot holds at most 256 rows: only the 256-row halves that exist are numbered
    t.n_small = t.n_vblocks * (2 * (t.big_tiles_m - 1) + 1) * t.tiles_n;
  }
  t.total_tiles = t.n_big + t.n_small + t.n_quarter;
  return t;
}

int launch_gemm(const GemmLaunch& L, cudaStream_t stream) {
  static thread_local GemmParams p;
  // an activation goes with the plain store only (the ring read-modify-write adds partial sums)
  if (L.activation != ACT_NONE && L.epilogue != EPI_STORE) return COMPASS_ERR_INVALID_ARG;
  if (L.epilogue != EPI_STORE && L.ring_scratch == nullptr) return COMPASS_ERR_INVALID_ARG;
  if (L.activation == ACT_SWIGLU && (L.N % 16 != 0 || L.ldo < L.N / 2)) return COMPASS_ERR_INVALID_ARG;
  DeviceInfo* info = nullptr;
  int st = device_info(&info);
  if (st != COMPASS_OK) return st;
  const TilePlan tiling = plan_tiles(L, info->max_pairs);
  const bool pair = tiling.pair != 0;
  const int b_box_rows = pair ? BN / 2 : BN;
  for (int i = 0; i < L.n_a; ++i)
    if (!encode_kmajor(&p.a_maps[i], L.a_ptr[i], L.a_map_rows[i] ? L.a_map_rows[i] : L.a_rows, L.K, BM))
      return record_cuda_error(cudaErrorUnknown);
  for (int i = 0; i < L.n_b; ++i)
    if (L.b_mn_major ? !encode_kmajor(&p.b_maps[i], L.b_ptr[i], L.K, L.N, 64)      // [K][N]: boxes of 64 columns x 64 k-rows
                     : !encode_kmajor(&p.b_maps[i], L.b_ptr[i], L.N, L.K, b_box_rows))
      return record_cuda_error(cudaErrorUnknown);
  for (int i = 0; i < L.n_out; ++i) {
    p.out[i] = static_cast<__nv_bfloat16*>(L.out_ptr[i]);
  }
  p.ring_scratch = static_cast<uint8_t*>(L.ring_scratch);
  p.ldo = L.ldo;
  p.n_blocks = L.n_blocks;
  p.rows_per_block = L.rows_per_block;
  p.N = int32_t(L.N);
  p.n_seg = L.n_seg;
  const int stage_k = pair ? 2 * BK : BK;      // Cfg<pair>::kStageK
  p.kb_per_seg = int32_t((L.K + stage_k - 1) / stage_k);
  const int64_t k_tail = L.K - int64_t(p.kb_per_seg - 1) * stage_k;
  p.tail_ksteps = int32_t((k_tail + UMMA_K - 1) / UMMA_K);
  p.group = tiling.group;
  p.sub_pad = tiling.sub_pad;
  p.vrows = tiling.vrows;
  p.frags_m = tiling.sub_pad / BM;
  p.tiles_m = tiling.tiles_m;
  p.tiles_n = tiling.tiles_n;
  p.total_tiles = tiling.total_tiles;
  p.epilogue = L.epilogue;
  p.last_step = L.last_step;
  p.wait_limit_us = L.wait_limit_us ? L.wait_limit_us : (default_wait_limit_us() ? default_wait_limit_us() : 2000000u);
  p.prefetch_stages = L.prefetch_stages;
  p.activation = L.activation;
  p.b_mn_major = L.b_mn_major ? 1 : 0;
  p.skew = L.skew < 0 ? 0 : (L.skew > 4 ? 4 : L.skew);
  p.a_hint = L.a_hint;
  p.b_hint = L.b_hint;

  p.status = L.status;
  p.tile_counters = L.tile_counters;
  p.flags = L.flags;
  p.flag_token = L.flag_token;
  for (int b = 0; b < L.n_blocks; ++b) p.blocks[b] = L.blocks[b];
  p.seg_strided = (L.seg_strided && L.n_seg > 1) ? 1 : 0;
  p.n_ranks = L.n_ranks > 0 ? L.n_ranks : 1;
  if (L.n_seg > 1 && !p.seg_strided) {
    if (L.n_blocks > kMaxSegBlocks) return COMPASS_ERR_UNSUPPORTED;
    for (int b = 0; b < L.n_blocks; ++b)
      for (int s = 0; s < L.n_seg; ++s) p.seg_rank[b][s] = L.seg_rank[b][s];
  }

  if (p.total_tiles <= 0) return COMPASS_OK;
  const bool mixed = tiling.mixed != 0;
  if (mixed) {
    p.big_tiles_m = tiling.big_tiles_m;
    p.n_big = tiling.n_big;
    p.n_small_end = tiling.n_big + tiling.n_small;
    p.h_last = tiling.h_last;
    p.kb_big = int32_t((L.K + BK - 1) / BK);
    p.tail_big = int32_t((L.K - int64_t(p.kb_big - 1) * BK + UMMA_K - 1) / UMMA_K);
    if (tiling.n_quarter > 0 && !L.b_mn_major)
      for (int i = 0; i < L.n_b; ++i)
        if (!encode_kmajor(&p.b_maps_q[i], L.b_ptr[i], L.N, L.K, BN / 4)) return record_cuda_error(cudaErrorUnknown);
  }
  cudaError_t e;
  if (pair) {
    const int pairs = p.total_tiles < info->max_pairs ? p.total_tiles : info->max_pairs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(2 * pairs));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = mixed ? kMixedSmemBytes : smem_bytes<true>();
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (mixed && L.activation != ACT_NONE) e = cudaLaunchKernelEx(&cfg, gemm_mixed_kernel<true>, p);
    else if (mixed) e = cudaLaunchKernelEx(&cfg, gemm_mixed_kernel<false>, p);
    else if (L.epilogue == EPI_RING_RMW_F32) e = cudaLaunchKernelEx(&cfg, gemm_kernel<true, false, true>, p);
    else if (L.activation != ACT_NONE) e = cudaLaunchKernelEx(&cfg, gemm_kernel<true, true, false>, p);
    else e = cudaLaunchKernelEx(&cfg, gemm_kernel<true, false, false>, p);
  } else {
    const int grid = p.total_tiles < info->num_sms ? p.total_tiles : info->num_sms;
    if (L.epilogue == EPI_RING_RMW_F32) gemm_kernel<false, false, true><<<grid, kThreads, smem_bytes<false>(), stream>>>(p);
    else if (L.activation != ACT_NONE) gemm_kernel<false, true, false><<<grid, kThreads, smem_bytes<false>(), stream>>>(p);
    else gemm_kernel<false, false, false><<<grid, kThreads, smem_bytes<false>(), stream>>>(p);
    e = cudaGetLastError();
  }
  count_kernel_launch();
  if (e != cudaSuccess) return record_cuda_error(e);
  e = cudaGetLastError();
  if (e != cudaSuccess) return record_cuda_error(e);
  return COMPASS_OK;
}

}  // namespace compass
