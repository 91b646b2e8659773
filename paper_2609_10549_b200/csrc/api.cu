// C ABI entry points: argument checks, mapping of the ring schedule onto GEMM
// launches, the InterDecom stream pipeline, workspace layout.
#include <atomic>
#include <cstring>
#include <mutex>

#include "internal.h"

namespace compass {

namespace {

std::atomic<int> g_last_cuda_error{0};
std::atomic<uint64_t> g_kernel_launches{0};
std::atomic<uint32_t> g_wait_limit_us{0};
std::atomic<int> g_drop_flag_writes{0};      // host-side failure injection: readiness-flag writes still to be left out

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate_problem(const compass_problem* pr, int want_op, bool need_d) {
  if (pr == nullptr) return COMPASS_ERR_INVALID_ARG;
  if (pr->op != COMPASS_OP_AG_GEMM && pr->op != COMPASS_OP_GEMM_RS) return COMPASS_ERR_INVALID_ARG;
  if (want_op >= 0 && pr->op != want_op) return COMPASS_ERR_INVALID_ARG;
  if (pr->P < 1 || (pr->rings != 1 && pr->rings != 2)) return COMPASS_ERR_INVALID_ARG;
  if (need_d && pr->d < 1) return COMPASS_ERR_INVALID_ARG;
  if (pr->order != COMPASS_ORDER_RANK_MAJOR && pr->order != COMPASS_ORDER_STEP_MAJOR) return COMPASS_ERR_INVALID_ARG;
  if (pr->copy_mode != COMPASS_COPY_KERNEL && pr->copy_mode != COMPASS_COPY_ENGINES) return COMPASS_ERR_INVALID_ARG;
  if (pr->op == COMPASS_OP_GEMM_RS && pr->rs_variant != COMPASS_RS_SEGMENTED_K && pr->rs_variant != COMPASS_RS_RING_RMW &&
      pr->rs_variant != COMPASS_RS_RING_RMW_F32)
    return COMPASS_ERR_INVALID_ARG;
  if (pr->b_layout != COMPASS_B_NK && pr->b_layout != COMPASS_B_KN) return COMPASS_ERR_INVALID_ARG;
  if (pr->ring_group != 0 && pr->ring_group != 1) {
    // contributors fused per read-modify-write pass: ring variants only, a divisor of P
    if (pr->op != COMPASS_OP_GEMM_RS || pr->rs_variant == COMPASS_RS_SEGMENTED_K) return COMPASS_ERR_INVALID_ARG;
    if (pr->ring_group < 2 || pr->P < 1 || pr->ring_group > pr->P || pr->P % pr->ring_group != 0) return COMPASS_ERR_INVALID_ARG;
  }
  if (pr->dtype != COMPASS_DTYPE_BF16 || pr->P > COMPASS_MAX_P) return COMPASS_ERR_UNSUPPORTED;
  if (pr->M <= 0 || pr->N <= 0 || pr->K <= 0) return COMPASS_ERR_SHAPE;
  if (pr->M % pr->P != 0 || (pr->M / pr->P) % pr->rings != 0) return COMPASS_ERR_SHAPE;
  if (need_d && (pr->M / pr->P) % pr->d != 0) return COMPASS_ERR_SHAPE;
  if (pr->K % 8 != 0 || pr->N % 8 != 0) return COMPASS_ERR_ALIGNMENT;
  if (pr->M > (1 << 30) || pr->N > (1 << 30) || pr->K > (1 << 30)) return COMPASS_ERR_UNSUPPORTED;
  return COMPASS_OK;
}

int validate_pointers(const void* const* a, const void* const* b, void* const* o, int P) {
  if (a == nullptr || b == nullptr || o == nullptr) return COMPASS_ERR_INVALID_ARG;
  for (int r = 0; r < P; ++r)
    if (a[r] == nullptr || b[r] == nullptr || o[r] == nullptr) return COMPASS_ERR_INVALID_ARG;
  for (int r = 0; r < P; ++r)
    if (!aligned16(a[r]) || !aligned16(b[r]) || !aligned16(o[r])) return COMPASS_ERR_ALIGNMENT;
  return COMPASS_OK;
}

int validate_workspace(const compass_problem* pr, int which, void* ws, size_t ws_bytes) {
  size_t need = 0;
  int st = compass_workspace_bytes(pr, which, &need);
  if (st != COMPASS_OK) return st;
  if (ws == nullptr) return COMPASS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0) return COMPASS_ERR_ALIGNMENT;
  if (ws_bytes < need) return COMPASS_ERR_BUFFER_TOO_SMALL;
  return COMPASS_OK;
}

inline int tiles_of(int64_t rows, int tile) { return int((rows + tile - 1) / tile); }

// Number of ring-RMW tile counters of a fused GEMM+ReduceScatter launch.
size_t rmw_counter_count(const compass_problem* pr) {
  const int64_t h = pr->M / pr->P / pr->rings;
  return size_t(pr->rings) * size_t(pr->P) * size_t(tiles_of(h, BM)) * size_t(tiles_of(pr->N, BN));
}

// Readiness flags of the push variant: one per (rank, partition).
size_t push_flag_count(const compass_problem* pr) { return size_t(pr->P) * size_t(pr->rings) * size_t(pr->P); }

// ---- fused launches: schedule -> blocks -------------------------------------

// AllGather+GEMM: one block per schedule entry.  Rank-major lists the table's own order; step-major lists
// step, then rank, then ring.  Either way every rank's blocks appear in its schedule order.
void plan_ag(const compass_problem* pr, const compass_sched_entry* table, GemmLaunch* L, compass_plan_block* view) {
  const int P = pr->P, rings = pr->rings;
  const int64_t m = pr->M / P;
  L->n_a = L->n_b = L->n_out = P;
  L->a_rows = m;
  L->K = pr->K;
  L->N = pr->N;
  L->ldo = pr->N;
  L->n_seg = 1;
  L->rows_per_block = int(m / rings);
  L->epilogue = EPI_STORE;
  int n = 0;
  const bool rank_major = pr->order == COMPASS_ORDER_RANK_MAJOR;
  // Runs of consecutive blocks that read the same weight shard: rank-major, all of a rank's entries; step-major, the
  // ring entries of one step of a rank.  Partitions below 256 rows are tiled in groups out of such a run (with two
  // rings: the two entries of one step, one CTA of a pair on each).
  L->share_run = rank_major ? rings * P : rings;
  const int n_entries = P * P * rings;
  for (int i = 0; i < n_entries; ++i) {
    // rank-major: the table's own order; step-major: step, then rank, then ring (a rank's entries of one step adjacent)
    const int rank = rank_major ? i / (P * rings) : (i / rings) % P;
    const int step = rank_major ? (i / rings) % P : i / (rings * P);
    const int ring = i % rings;
    const compass_sched_entry& e = table[(size_t(rank) * P + step) * rings + ring];
    BlockDesc& b = L->blocks[n];
    std::memset(&b, 0, sizeof(b));
    b.a_map = uint8_t(e.chunk);                       // read the owner's shard: gather by address
    b.a_row0 = e.row_begin - e.chunk * int32_t(m);
    b.b_map = uint8_t(rank);
    b.out_idx = uint8_t(rank);
    b.out_row0 = e.row_begin;
    b.step = uint8_t(step);
    b.part = uint8_t(e.part);
    if (view) {
      compass_plan_block& v = view[n];
      v.rank = rank; v.step = step; v.ring = ring; v.part = e.part;
      v.a_tensor = e.chunk; v.a_row_begin = b.a_row0;
      v.out_tensor = rank; v.out_row_begin = b.out_row0;
      v.rows = e.row_count;
    }
    ++n;
  }
  L->n_blocks = n;
}

// GEMM+ReduceScatter, segmented K: one block per partition; segment s of the
// k-loop reads the rank that contributes at step s of the ring.
void plan_rs_segmented(const compass_problem* pr, const compass_sched_entry* table, GemmLaunch* L,
                       compass_plan_block* view) {
  const int P = pr->P, rings = pr->rings;
  const int64_t m = pr->M / P;
  const int64_t h = m / rings;
  L->n_a = L->n_b = L->n_out = P;
  L->a_rows = pr->M;
  L->K = pr->K;
  L->N = pr->N;
  L->ldo = pr->N;
  L->n_seg = P;
  L->rows_per_block = int(h);
  L->share_run = 1;      // every partition walks the ranks' K slices in its own ring order: no two blocks share a B tile
  L->epilogue = EPI_STORE;
  const int n_parts = rings * P;
  for (int part = 0; part < n_parts; ++part) {
    const int chunk = part / rings, ring = part % rings;
    BlockDesc& b = L->blocks[part];
    std::memset(&b, 0, sizeof(b));
    b.a_row0 = int32_t(chunk * m + ring * h);
    b.out_idx = uint8_t(chunk);
    b.out_row0 = int32_t(ring * h);
    b.step = uint8_t(P - 1);
    b.part = uint8_t(part);
    if (view) {
      compass_plan_block& v = view[part];
      v.rank = -1; v.step = P - 1; v.ring = ring; v.part = part;
      v.a_tensor = -1; v.a_row_begin = b.a_row0;
      v.out_tensor = chunk; v.out_row_begin = b.out_row0;
      v.rows = int32_t(h);
    }
  }
  for (int rank = 0; rank < P; ++rank)
    for (int step = 0; step < P; ++step)
      for (int ring = 0; ring < rings; ++ring) {
        const compass_sched_entry& e = table[(size_t(rank) * P + step) * rings + ring];
        L->seg_rank[e.part][step] = uint8_t(rank);
      }
  L->n_blocks = n_parts;
}

// GEMM+ReduceScatter, ring read-modify-write: one block per schedule entry in
// the same launch order as AllGather+GEMM; contributor `step` of a partition
// precedes contributor step+1 in the launch.
void plan_rs_ring(const compass_problem* pr, const compass_sched_entry* table, GemmLaunch* L, compass_plan_block* view) {
  const int P = pr->P, rings = pr->rings;
  const int64_t m = pr->M / P;
  L->n_a = L->n_b = L->n_out = P;
  L->a_rows = pr->M;
  L->K = pr->K;
  L->N = pr->N;
  L->ldo = pr->N;
  L->n_seg = 1;
  L->rows_per_block = int(m / rings);
  L->share_run = rings;  // a rank's two ring entries of one step are adjacent and multiply by the same B_rank
  L->epilogue = pr->rs_variant == COMPASS_RS_RING_RMW_F32 ? EPI_RING_RMW_F32 : EPI_RING_RMW;
  L->last_step = P - 1;
  L->seg_strided = false;
  L->n_ranks = P;
  const int G = pr->ring_group > 1 ? pr->ring_group : 1;
  if (G > 1) {
    // G consecutive contributors of a partition share a tile: its k-loop runs over their K slices in ring order.
    // The contributors of a partition follow one another along its ring, so the lead's neighbour (`peer`) gives the
    // stride between their ranks.
    L->n_seg = G;
    L->share_run = 1;
    L->seg_strided = true;
    L->last_step = P / G - 1;
  }
  int n = 0;
  bool consistent = true;
  for (int step = 0; step < P; step += G)
    for (int rank = 0; rank < P; ++rank)        // a rank's entries of one step are adjacent: they share its weight shard in L2
      for (int ring = 0; ring < rings; ++ring) {
        const compass_sched_entry& e = table[(size_t(rank) * P + step) * rings + ring];
        BlockDesc& b = L->blocks[n];
        std::memset(&b, 0, sizeof(b));
        b.a_map = uint8_t(rank);
        b.b_map = uint8_t(rank);
        b.seg_stride = uint8_t(G > 1 ? (e.peer - rank + P) % P : 0);
        for (int i = 1; i < G; ++i) {             // the table must agree: contributor step+i of this partition
          const int r_i = (rank + i * int(b.seg_stride)) % P;
          if (table[(size_t(r_i) * P + step + i) * rings + ring].part != e.part) consistent = false;
        }
        b.a_row0 = e.row_begin;
        b.out_idx = uint8_t(e.chunk);
        b.out_row0 = e.row_begin - e.chunk * int32_t(m);
        b.step = uint8_t(step / G);
        b.part = uint8_t(e.part);
        if (view) {
          compass_plan_block& v = view[n];      // grouped: the lead contributor's rank and step
          v.rank = rank; v.step = step; v.ring = ring; v.part = e.part;
          v.a_tensor = rank; v.a_row_begin = b.a_row0;
          v.out_tensor = e.chunk; v.out_row_begin = b.out_row0;
          v.rows = e.row_count;
        }
        ++n;
      }
  L->n_blocks = consistent ? n : -1;
}

int plan_fused(const compass_problem* pr, GemmLaunch* L, compass_plan_block* view) {
  static thread_local compass_sched_entry table[kMaxBlocks];
  int st = validate_schedule_args(pr->op, pr->P, pr->rings, pr->M);
  if (st != COMPASS_OK) return st;
  build_schedule(pr->op, pr->P, pr->rings, pr->M, table);
  L->seg_strided = false;
  if (pr->op == COMPASS_OP_AG_GEMM) plan_ag(pr, table, L, view);
  else if (pr->rs_variant == COMPASS_RS_SEGMENTED_K) plan_rs_segmented(pr, table, L, view);
  else plan_rs_ring(pr, table, L, view);
  if (L->n_blocks < 0) return COMPASS_ERR_UNSUPPORTED;     // (a schedule whose contributors do not follow the ring)
  L->b_mn_major = pr->b_layout == COMPASS_B_KN;
  if (view) {
    const int per_block = tiles_of(L->rows_per_block, gemm_tile_rows(L->mode, L->rows_per_block)) * tiles_of(L->N, BN);
    for (int i = 0; i < L->n_blocks; ++i) {
      view[i].first_tile = i * per_block;
      view[i].tile_count = per_block;
    }
  }
  return COMPASS_OK;
}

// Running sums of the ring read-modify-write variants: behind the tile counters, one 128 x 256 fragment per counter
// (BF16 or FP32), in the order the epilogue's lanes hold them.
size_t ring_scratch_bytes(const compass_problem* pr) {
  if (pr->op != COMPASS_OP_GEMM_RS || pr->rs_variant == COMPASS_RS_SEGMENTED_K) return 0;
  const size_t element = pr->rs_variant == COMPASS_RS_RING_RMW_F32 ? sizeof(float) : 2;
  return rmw_counter_count(pr) * size_t(BM) * size_t(BN) * element;
}

void set_running_sums(const compass_problem* pr, GemmLaunch* L, void* ws) {
  L->ring_scratch = nullptr;
  if (ring_scratch_bytes(pr) == 0) return;
  L->ring_scratch = static_cast<uint8_t*>(ws) + COMPASS_STATUS_BYTES + align_up(rmw_counter_count(pr) * sizeof(int32_t));
}

int fused_call(const compass_problem* pr, int op, const void* const* A, const void* const* B, void* const* out, void* ws,
               size_t ws_bytes, void* stream) {
  int st = validate_problem(pr, op, false);
  if (st != COMPASS_OK) return st;
  st = validate_pointers(A, B, out, pr->P);
  if (st != COMPASS_OK) return st;
  st = validate_workspace(pr, COMPASS_WS_FUSED, ws, ws_bytes);
  if (st != COMPASS_OK) return st;
  static thread_local GemmLaunch L;
  st = plan_fused(pr, &L, nullptr);
  if (st != COMPASS_OK) return st;
  for (int r = 0; r < pr->P; ++r) {
    L.a_ptr[r] = A[r];
    L.b_ptr[r] = B[r];
    L.out_ptr[r] = out[r];
  }
  L.status = static_cast<StatusBlock*>(ws);
  L.tile_counters = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + COMPASS_STATUS_BYTES);
  set_running_sums(pr, &L, ws);
  return launch_gemm(L, static_cast<cudaStream_t>(stream));
}

// ---- MLP block -----------------------------------------------------------------

// The two fused operators of the block as problems of their own.
int mlp_problems(const compass_mlp* mp, compass_problem* ag, compass_problem* rs) {
  if (mp == nullptr) return COMPASS_ERR_INVALID_ARG;
  if (mp->activation != COMPASS_ACT_NONE && mp->activation != COMPASS_ACT_GELU_TANH && mp->activation != COMPASS_ACT_SWIGLU)
    return COMPASS_ERR_INVALID_ARG;
  if (mp->b_layout != COMPASS_B_NK && mp->b_layout != COMPASS_B_KN) return COMPASS_ERR_INVALID_ARG;
  if (mp->hidden <= 0 || mp->ffn <= 0) return COMPASS_ERR_SHAPE;
  // SwiGLU: (gate, up) column pairs; the result's rows must still be a multiple of 16 bytes for the second GEMM's loads
  if (mp->activation == COMPASS_ACT_SWIGLU && mp->ffn % 16 != 0) return COMPASS_ERR_ALIGNMENT;
  std::memset(ag, 0, sizeof(*ag));
  ag->op = COMPASS_OP_AG_GEMM;
  ag->P = mp->P;
  ag->rings = mp->rings;
  ag->d = 1;
  ag->M = mp->M;
  ag->N = mp->ffn;
  ag->K = mp->hidden;
  ag->dtype = COMPASS_DTYPE_BF16;
  ag->rs_variant = COMPASS_RS_SEGMENTED_K;
  ag->order = mp->order;
  ag->copy_mode = COMPASS_COPY_KERNEL;
  ag->b_layout = mp->b_layout;
  *rs = *ag;
  rs->op = COMPASS_OP_GEMM_RS;
  rs->N = mp->hidden;
  rs->K = mp->activation == COMPASS_ACT_SWIGLU ? mp->ffn / 2 : mp->ffn;
  rs->rs_variant = mp->rs_variant;
  int st = validate_problem(ag, COMPASS_OP_AG_GEMM, false);
  if (st != COMPASS_OK) return st;
  return validate_problem(rs, COMPASS_OP_GEMM_RS, false);
}


// ---- InterDecom ----------------------------------------------------------------

// Events that order the two streams of a call; created on first use, one set per device
// (an event belongs to the device that was current when it was created).
struct EventPool {
  static constexpr int kMaxDevices = 64;
  std::mutex mu;
  cudaEvent_t all[kMaxDevices][2 * 16 + 2];
  int made[kMaxDevices] = {};
  cudaEvent_t* ev = nullptr;      // the current device's set, valid after ensure()
  cudaStream_t side_stream[kMaxDevices] = {};   // second copy stream of the push variant, created on first use
  // A non-blocking stream of the library's own on the current device (under `mu`).
  int ensure_side_stream(cudaStream_t* out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return COMPASS_ERR_UNSUPPORTED;
    if (side_stream[dev] == nullptr) {
      e = cudaStreamCreateWithFlags(&side_stream[dev], cudaStreamNonBlocking);
      if (e != cudaSuccess) return record_cuda_error(e);
    }
    *out = side_stream[dev];
    return COMPASS_OK;
  }
  int ensure(int n) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return COMPASS_ERR_UNSUPPORTED;
    while (made[dev] < n) {
      e = cudaEventCreateWithFlags(&all[dev][made[dev]], cudaEventDisableTiming);
      if (e != cudaSuccess) return record_cuda_error(e);
      ++made[dev];
    }
    ev = all[dev];
    return COMPASS_OK;
  }
};
EventPool g_events;

// comm_only: enqueue the sub-collectives alone (the T_comm of Section IV-C), without the sub-GEMMs.
int decomp_ag(const compass_problem* pr, const void* const* A, const void* const* B, void* const* C, uint8_t* ws,
              cudaStream_t s_comp, cudaStream_t s_copy, cudaEvent_t* ev, bool comm_only) {
  const int P = pr->P, d = pr->d;
  const int64_t m = pr->M / P, K = pr->K, sl = m / d;
  const size_t gather_bytes = align_up(size_t(pr->M) * size_t(K) * 2);
  uint8_t* G[kMaxP];
  for (int r = 0; r < P; ++r) G[r] = ws + COMPASS_STATUS_BYTES + size_t(r) * gather_bytes;

  static thread_local GemmLaunch L;
  L.n_a = L.n_b = L.n_out = P;
  L.b_mn_major = pr->b_layout == COMPASS_B_KN;
  L.a_rows = pr->M;
  L.K = K;
  L.N = pr->N;
  L.ldo = pr->N;
  L.n_seg = 1;
  L.rows_per_block = int(sl);
  L.share_run = P;       // rank r's P row slices are adjacent and multiply by B_r
  L.epilogue = EPI_STORE;
  L.status = reinterpret_cast<StatusBlock*>(ws);
  L.tile_counters = nullptr;
  for (int r = 0; r < P; ++r) {
    L.a_ptr[r] = G[r];
    L.b_ptr[r] = B[r];
    L.out_ptr[r] = C[r];
  }
  cudaError_t e;
  // the copy stream starts after whatever precedes this call on the compute stream
  if ((e = cudaEventRecord(ev[0], s_comp)) != cudaSuccess) return record_cuda_error(e);
  if ((e = cudaStreamWaitEvent(s_copy, ev[0], 0)) != cudaSuccess) return record_cuda_error(e);
  for (int j = 0; j < d; ++j) {
    // sub-AllGather j: row slice j of every shard into every rank's gather buffer
    if (pr->copy_mode == COMPASS_COPY_ENGINES) {
      for (int r = 0; r < P; ++r)
        for (int q = 0; q < P; ++q) {
          const uint8_t* src = static_cast<const uint8_t*>(A[q]) + size_t(j * sl) * size_t(K) * 2;
          uint8_t* dst = G[r] + size_t(q * m + j * sl) * size_t(K) * 2;
          e = cudaMemcpyAsync(dst, src, size_t(sl) * size_t(K) * 2, cudaMemcpyDeviceToDevice, s_copy);
          if (e != cudaSuccess) return record_cuda_error(e);
        }
    } else {
      void* gptr[kMaxP];
      for (int r = 0; r < P; ++r) gptr[r] = G[r];
      int stg = launch_gather_slices(A, gptr, P, m, K, j * sl, sl, s_copy);
      if (stg != COMPASS_OK) return stg;
    }
    if ((e = cudaEventRecord(ev[1 + j], s_copy)) != cudaSuccess) return record_cuda_error(e);
    if ((e = cudaStreamWaitEvent(s_comp, ev[1 + j], 0)) != cudaSuccess) return record_cuda_error(e);
    if (comm_only) continue;
    // sub-GEMM j on the gathered rows
    // rank-major, like the fused launch: a rank's weight shard stays in L2 across its P row slices
    int n = 0;
    for (int r = 0; r < P; ++r)
      for (int q = 0; q < P; ++q) {
        BlockDesc& b = L.blocks[n++];
        std::memset(&b, 0, sizeof(b));
        b.a_map = uint8_t(r);
        b.b_map = uint8_t(r);
        b.out_idx = uint8_t(r);
        b.a_row0 = int32_t(q * m + j * sl);
        b.out_row0 = b.a_row0;
      }
    L.n_blocks = n;
    int st = launch_gemm(L, s_comp);
    if (st != COMPASS_OK) return st;
  }
  return COMPASS_OK;
}

int decomp_rs(const compass_problem* pr, const void* const* A, const void* const* B, void* const* Out, uint8_t* ws,
              cudaStream_t s_comp, cudaStream_t s_copy, cudaEvent_t* ev, bool comm_only) {
  const int P = pr->P, d = pr->d;
  const int64_t m = pr->M / P, sl = m / d;
  const size_t partial_bytes = align_up(size_t(pr->M) * size_t(pr->N) * 2);
  void* W[kMaxP];
  for (int q = 0; q < P; ++q) W[q] = ws + COMPASS_STATUS_BYTES + size_t(q) * partial_bytes;

  static thread_local GemmLaunch L;
  L.n_a = L.n_b = L.n_out = P;
  L.b_mn_major = pr->b_layout == COMPASS_B_KN;
  L.a_rows = pr->M;
  L.K = pr->K;
  L.N = pr->N;
  L.ldo = pr->N;
  L.n_seg = 1;
  L.rows_per_block = int(sl);
  L.share_run = P;       // rank q's P row slices (one per owner) are adjacent and multiply by B_q
  L.epilogue = EPI_STORE;
  L.status = reinterpret_cast<StatusBlock*>(ws);
  L.tile_counters = nullptr;
  for (int q = 0; q < P; ++q) {
    L.a_ptr[q] = A[q];
    L.b_ptr[q] = B[q];
    L.out_ptr[q] = W[q];
  }
  cudaError_t e;
  for (int j = 0; j < d; ++j) {
    // sub-GEMM j: every rank's partial rows of slice j of every owner's block
    // rank-major: rank q's weight shard stays in L2 across the P owners' row slices
    int n = 0;
    for (int q = 0; q < P; ++q)
      for (int c = 0; c < P; ++c) {
        BlockDesc& b = L.blocks[n++];
        std::memset(&b, 0, sizeof(b));
        b.a_map = uint8_t(q);
        b.b_map = uint8_t(q);
        b.out_idx = uint8_t(q);
        b.a_row0 = int32_t(c * m + j * sl);
        b.out_row0 = b.a_row0;
      }
    L.n_blocks = n;
    int st = comm_only ? int(COMPASS_OK) : launch_gemm(L, s_comp);
    if (st != COMPASS_OK) return st;
    if ((e = cudaEventRecord(ev[1 + j], s_comp)) != cudaSuccess) return record_cuda_error(e);
    if ((e = cudaStreamWaitEvent(s_copy, ev[1 + j], 0)) != cudaSuccess) return record_cuda_error(e);
    // sub-ReduceScatter j
    st = launch_reduce_partials(W, P, Out, m, pr->N, j * sl, sl, s_copy);
    if (st != COMPASS_OK) return st;
  }
  // later work on the compute stream sees the reduced output
  if ((e = cudaEventRecord(ev[0], s_copy)) != cudaSuccess) return record_cuda_error(e);
  if ((e = cudaStreamWaitEvent(s_comp, ev[0], 0)) != cudaSuccess) return record_cuda_error(e);
  return COMPASS_OK;
}

}  // namespace

int record_cuda_error(cudaError_t e) {
  g_last_cuda_error.store(int(e));
  return COMPASS_ERR_CUDA;
}
void count_kernel_launch() { g_kernel_launches.fetch_add(1, std::memory_order_relaxed); }
uint32_t default_wait_limit_us() { return g_wait_limit_us.load(std::memory_order_relaxed); }

}  // namespace compass

using namespace compass;

extern "C" int compass_workspace_bytes(const compass_problem* pr, int which, size_t* bytes) {
  if (bytes == nullptr) return COMPASS_ERR_INVALID_ARG;
  if (which != COMPASS_WS_FUSED && which != COMPASS_WS_DECOMP && which != COMPASS_WS_PUSH) return COMPASS_ERR_INVALID_ARG;
  if (which == COMPASS_WS_PUSH && pr != nullptr && pr->op != COMPASS_OP_AG_GEMM) return COMPASS_ERR_INVALID_ARG;
  int st = validate_problem(pr, -1, which == COMPASS_WS_DECOMP);
  if (st != COMPASS_OK) return st;
  size_t total = COMPASS_STATUS_BYTES;
  if (which == COMPASS_WS_FUSED) {
    if (pr->op == COMPASS_OP_GEMM_RS && pr->rs_variant != COMPASS_RS_SEGMENTED_K)
      total += align_up(rmw_counter_count(pr) * sizeof(int32_t));
    total += align_up(ring_scratch_bytes(pr));
  } else if (which == COMPASS_WS_DECOMP) {
    const size_t inner = pr->op == COMPASS_OP_AG_GEMM ? size_t(pr->K) : size_t(pr->N);
    total += size_t(pr->P) * align_up(size_t(pr->M) * inner * 2);
  } else {
    total += align_up(push_flag_count(pr) * sizeof(uint32_t));
    total += size_t(pr->P) * align_up(size_t(pr->M) * size_t(pr->K) * 2);
  }
  *bytes = total;
  return COMPASS_OK;
}

extern "C" int compass_workspace_init(void* ws, size_t ws_bytes, void* stream) {
  if (ws == nullptr || ws_bytes < COMPASS_STATUS_BYTES) return COMPASS_ERR_INVALID_ARG;
  cudaError_t e = cudaMemsetAsync(ws, 0, ws_bytes, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return record_cuda_error(e);
  return COMPASS_OK;
}

extern "C" int compass_read_status(void* ws, void* stream, int* detail) {
  if (ws == nullptr) return COMPASS_ERR_INVALID_ARG;
  StatusBlock host;
  cudaError_t e = cudaMemcpyAsync(&host, ws, sizeof(host), cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return record_cuda_error(e);
  e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return record_cuda_error(e);
  if (detail) *detail = host.detail;
  return host.code;
}

extern "C" int compass_read_kernel_clock(void* ws, void* stream, uint64_t* sm_cycles, uint64_t* nanoseconds) {
  if (ws == nullptr || sm_cycles == nullptr || nanoseconds == nullptr) return COMPASS_ERR_INVALID_ARG;
  StatusBlock host;
  cudaError_t e = cudaMemcpyAsync(&host, ws, sizeof(host), cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return record_cuda_error(e);
  e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return record_cuda_error(e);
  *sm_cycles = host.kernel_cycles;
  *nanoseconds = host.kernel_ns;
  return COMPASS_OK;
}

extern "C" int compass_launch_plan(const compass_problem* pr, compass_plan_block* out, size_t capacity, size_t* count) {
  if (count == nullptr) return COMPASS_ERR_INVALID_ARG;
  int st = validate_problem(pr, -1, false);
  if (st != COMPASS_OK) return st;
  const bool per_entry = pr->op == COMPASS_OP_AG_GEMM || pr->rs_variant != COMPASS_RS_SEGMENTED_K;
  const int group = (pr->op == COMPASS_OP_GEMM_RS && pr->ring_group > 1) ? pr->ring_group : 1;   // contributors per block
  const size_t n = size_t(pr->rings) * pr->P * (per_entry ? pr->P / group : 1);
  *count = n;
  if (out == nullptr) return COMPASS_OK;
  if (capacity < n) return COMPASS_ERR_BUFFER_TOO_SMALL;
  static thread_local GemmLaunch L;
  static thread_local compass_plan_block view[kMaxBlocks];
  st = plan_fused(pr, &L, view);
  if (st != COMPASS_OK) return st;
  std::memcpy(out, view, n * sizeof(compass_plan_block));
  return COMPASS_OK;
}

extern "C" int compass_tile_plan(const compass_problem* pr, int decomposed, int cta_pairs, compass_tile_counts* out) {
  if (out == nullptr || cta_pairs < 0) return COMPASS_ERR_INVALID_ARG;
  int st = validate_problem(pr, -1, decomposed != 0);
  if (st != COMPASS_OK) return st;
  static thread_local GemmLaunch L;
  if (decomposed) {
    // one sub-GEMM of compass_decomp: P x P blocks of (M/P)/d rows, a rank's P blocks adjacent
    if (pr->d > 16) return COMPASS_ERR_UNSUPPORTED;
    L = GemmLaunch{};
    L.n_blocks = pr->P * pr->P;
    L.rows_per_block = int(pr->M / pr->P / pr->d);
    L.share_run = pr->P;
    L.N = pr->N;
    L.K = pr->K;
  } else {
    L.mode = GEMM_MODE_AUTO;
    st = plan_fused(pr, &L, nullptr);
    if (st != COMPASS_OK) return st;
  }
  const TilePlan t = plan_tiles(L, cta_pairs);
  out->cta_pairs = t.pair;
  out->blocks = L.n_blocks;
  out->rows_per_block = L.rows_per_block;
  out->blocks_per_group = t.group;
  out->tiles_512x256 = t.mixed ? t.n_big : 0;
  out->tiles_256x256 = t.pair ? (t.mixed ? t.n_small : t.total_tiles) : 0;
  out->tiles_256x128 = t.mixed ? t.n_quarter : 0;
  out->tiles_128x256 = t.pair ? 0 : t.total_tiles;
  out->total_tiles = t.total_tiles;
  return COMPASS_OK;
}

extern "C" int compass_ag_gemm(const compass_problem* pr, const void* const* A, const void* const* B, void* const* C,
                               void* ws, size_t ws_bytes, void* stream) {
  return fused_call(pr, COMPASS_OP_AG_GEMM, A, B, C, ws, ws_bytes, stream);
}

extern "C" int compass_gemm_rs(const compass_problem* pr, const void* const* A, const void* const* B, void* const* Out,
                               void* ws, size_t ws_bytes, void* stream) {
  return fused_call(pr, COMPASS_OP_GEMM_RS, A, B, Out, ws, ws_bytes, stream);
}

// cuStreamWriteValue32: a stream-ordered 32-bit store executed by the front end (no SM, no copy engine).
typedef CUresult (*StreamWriteValue32Fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
static StreamWriteValue32Fn stream_write_fn() {
  // looked up once; the initialisation of a function-local static is thread-safe
  static const StreamWriteValue32Fn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      return reinterpret_cast<StreamWriteValue32Fn>(ptr);
    return static_cast<StreamWriteValue32Fn>(nullptr);
  }();
  return fn;
}

extern "C" int compass_mlp_workspace_bytes(const compass_mlp* mp, size_t* bytes) {
  if (bytes == nullptr) return COMPASS_ERR_INVALID_ARG;
  compass_problem ag, rs;
  int st = mlp_problems(mp, &ag, &rs);
  if (st != COMPASS_OK) return st;
  size_t a = 0, b = 0;
  st = compass_workspace_bytes(&ag, COMPASS_WS_FUSED, &a);
  if (st != COMPASS_OK) return st;
  st = compass_workspace_bytes(&rs, COMPASS_WS_FUSED, &b);
  if (st != COMPASS_OK) return st;
  *bytes = a > b ? a : b;      // the two launches are ordered on one stream and share status block and counters
  return COMPASS_OK;
}

extern "C" int compass_mlp_block(const compass_mlp* mp, const void* const* X, const void* const* W0, void* const* H,
                                 const void* const* W1, void* const* Out, void* ws, size_t ws_bytes, void* stream) {
  compass_problem ag, rs;
  int st = mlp_problems(mp, &ag, &rs);
  if (st != COMPASS_OK) return st;
  st = validate_pointers(X, W0, H, mp->P);
  if (st != COMPASS_OK) return st;
  st = validate_pointers(H, W1, Out, mp->P);
  if (st != COMPASS_OK) return st;
  size_t need = 0;
  st = compass_mlp_workspace_bytes(mp, &need);
  if (st != COMPASS_OK) return st;
  if (ws == nullptr) return COMPASS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0) return COMPASS_ERR_ALIGNMENT;
  if (ws_bytes < need) return COMPASS_ERR_BUFFER_TOO_SMALL;

  static thread_local GemmLaunch L;
  // AllGather + GEMM0, the activation applied in the epilogue: H_r = act(gather(X) * W0_r)
  st = plan_fused(&ag, &L, nullptr);
  if (st != COMPASS_OK) return st;
  for (int r = 0; r < mp->P; ++r) {
    L.a_ptr[r] = X[r];
    L.b_ptr[r] = W0[r];
    L.out_ptr[r] = H[r];
  }
  L.activation = mp->activation;
  L.ldo = rs.K;                                  // H's row pitch: ffn, or ffn / 2 with SwiGLU
  L.status = static_cast<StatusBlock*>(ws);
  L.tile_counters = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + COMPASS_STATUS_BYTES);
  st = launch_gemm(L, static_cast<cudaStream_t>(stream));
  L.activation = ACT_NONE;                       // the launch descriptor is reused by the next call on this thread
  if (st != COMPASS_OK) return st;
  // GEMM1 + ReduceScatter on the stream-ordered result
  st = plan_fused(&rs, &L, nullptr);
  if (st != COMPASS_OK) return st;
  for (int r = 0; r < mp->P; ++r) {
    L.a_ptr[r] = H[r];
    L.b_ptr[r] = W1[r];
    L.out_ptr[r] = Out[r];
  }
  L.status = static_cast<StatusBlock*>(ws);
  L.tile_counters = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + COMPASS_STATUS_BYTES);
  set_running_sums(&rs, &L, ws);
  return launch_gemm(L, static_cast<cudaStream_t>(stream));
}

extern "C" int compass_ag_gemm_push(const compass_problem* pr, const void* const* A, const void* const* B, void* const* C,
                                    void* ws, size_t ws_bytes, void* stream_compute, void* stream_copy) {
  int st = validate_problem(pr, COMPASS_OP_AG_GEMM, false);
  if (st != COMPASS_OK) return st;
  st = validate_pointers(A, B, C, pr->P);
  if (st != COMPASS_OK) return st;
  st = validate_workspace(pr, COMPASS_WS_PUSH, ws, ws_bytes);
  if (st != COMPASS_OK) return st;
  if (stream_compute == stream_copy) return COMPASS_ERR_INVALID_ARG;
  StreamWriteValue32Fn write_value = stream_write_fn();
  if (write_value == nullptr) return COMPASS_ERR_UNSUPPORTED;

  const int P = pr->P, rings = pr->rings;
  const int64_t m = pr->M / P, h = m / rings, K = pr->K;
  uint8_t* base = static_cast<uint8_t*>(ws);
  uint32_t* flags = reinterpret_cast<uint32_t*>(base + COMPASS_STATUS_BYTES);
  const size_t gather_bytes = align_up(size_t(pr->M) * size_t(K) * 2);
  uint8_t* G[kMaxP];
  for (int r = 0; r < P; ++r)
    G[r] = base + COMPASS_STATUS_BYTES + align_up(push_flag_count(pr) * sizeof(uint32_t)) + size_t(r) * gather_bytes;

  static thread_local compass_sched_entry table[kMaxBlocks];
  build_schedule(COMPASS_OP_AG_GEMM, P, rings, pr->M, table);
  // A flag is up once it holds this call's token; tokens grow, so flags never need clearing.
  static std::atomic<uint32_t> epoch{0};
  const uint32_t token = epoch.fetch_add(1) + 1;

  static thread_local GemmLaunch L;
  L.n_a = 2 * P;                       // maps 0..P-1: the shards, P..2P-1: the gather buffers
  L.b_mn_major = pr->b_layout == COMPASS_B_KN;
  L.n_b = L.n_out = P;
  L.a_rows = m;
  L.K = K;
  L.N = pr->N;
  L.ldo = pr->N;
  L.n_seg = 1;
  L.rows_per_block = int(h);
  L.share_run = rings;
  L.epilogue = EPI_STORE;
  L.status = reinterpret_cast<StatusBlock*>(ws);
  L.flags = flags;
  L.flag_token = token;
  for (int r = 0; r < P; ++r) {
    L.a_ptr[r] = A[r];
    L.a_map_rows[r] = m;
    L.a_ptr[P + r] = G[r];
    L.a_map_rows[P + r] = pr->M;
    L.b_ptr[r] = B[r];
    L.out_ptr[r] = C[r];
  }
  int n = 0;
  for (int step = 0; step < P; ++step)
    for (int rank = 0; rank < P; ++rank)        // a rank's entries of one step are adjacent: they share its weight shard in L2
      for (int ring = 0; ring < rings; ++ring) {
        const compass_sched_entry& e = table[(size_t(rank) * P + step) * rings + ring];
        BlockDesc& b = L.blocks[n++];
        b = BlockDesc{};
        if (step == 0) {                       // local data: available at once
          b.a_map = uint8_t(rank);
          b.a_row0 = e.row_begin - e.chunk * int32_t(m);
        } else {                               // arrives in this rank's gather buffer
          b.a_map = uint8_t(P + rank);
          b.a_row0 = e.row_begin;
          b.flag1 = uint16_t(1 + rank * rings * P + e.part);
        }
        b.b_map = uint8_t(rank);
        b.out_idx = uint8_t(rank);
        b.out_row0 = e.row_begin;
        b.step = uint8_t(step);
        b.part = uint8_t(e.part);
      }
  L.n_blocks = n;

  cudaStream_t sc = static_cast<cudaStream_t>(stream_compute), sp = static_cast<cudaStream_t>(stream_copy);
  std::lock_guard<std::mutex> lock(g_events.mu);
  st = g_events.ensure(3);
  if (st != COMPASS_OK) return st;
  // The two rings move independent partitions (a partition travels along one ring only), so their copy chains
  // run on two streams: the caller's copy stream and one of the library's own.  One chain of 2(P-1)P small
  // copies, each followed by a flag write, would otherwise be what the GEMM waits for.
  cudaStream_t ring_stream[2] = {sp, sp};
  if (rings == 2) {
    st = g_events.ensure_side_stream(&ring_stream[1]);
    if (st != COMPASS_OK) return st;
  }
  cudaError_t e;
  // Inside a stream capture the token is frozen into the graph, so a replay would find the flags of the
  // previous replay already up: the captured work then starts by clearing them.
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if ((e = cudaStreamIsCapturing(sc, &capturing)) != cudaSuccess) return record_cuda_error(e);
  if (capturing == cudaStreamCaptureStatusActive &&
      (e = cudaMemsetAsync(flags, 0, push_flag_count(pr) * sizeof(uint32_t), sc)) != cudaSuccess)
    return record_cuda_error(e);
  // the pushes start after whatever precedes this call on the compute stream (inputs ready, buffers free)
  if ((e = cudaEventRecord(g_events.ev[0], sc)) != cudaSuccess) return record_cuda_error(e);
  if ((e = cudaStreamWaitEvent(sp, g_events.ev[0], 0)) != cudaSuccess) return record_cuda_error(e);
  if (rings == 2 && (e = cudaStreamWaitEvent(ring_stream[1], g_events.ev[0], 0)) != cudaSuccess) return record_cuda_error(e);
  // The kernel goes first: its step-0 tiles need nothing, and the host needs a while to enqueue the 2(P-1)P
  // copies and flag writes that follow (tiles of later steps wait, bounded, for their flags).
  st = launch_gemm(L, sc);
  if (st != COMPASS_OK) return st;
  const size_t part_bytes = size_t(h) * size_t(K) * 2;
  for (int step = 1; step < P; ++step)
    for (int ring = 0; ring < rings; ++ring)
      for (int rank = 0; rank < P; ++rank) {
        const compass_sched_entry& en = table[(size_t(rank) * P + step) * rings + ring];
        const int peer = en.peer;              // upstream neighbour that pushes the partition
        const uint8_t* src = (step == 1)
                                 ? static_cast<const uint8_t*>(A[peer]) + size_t(en.row_begin - en.chunk * m) * size_t(K) * 2
                                 : G[peer] + size_t(en.row_begin) * size_t(K) * 2;
        uint8_t* dst = G[rank] + size_t(en.row_begin) * size_t(K) * 2;
        cudaStream_t s = ring_stream[ring];
        if ((e = cudaMemcpyAsync(dst, src, part_bytes, cudaMemcpyDeviceToDevice, s)) != cudaSuccess)
          return record_cuda_error(e);
        uint32_t* flag = flags + size_t(rank) * rings * P + en.part;
        // failure injection for tests of the bounded flag wait: the copy is made, its flag is never raised
        if (g_drop_flag_writes.load(std::memory_order_relaxed) > 0 && g_drop_flag_writes.fetch_sub(1) > 0) continue;
        if (write_value(reinterpret_cast<CUstream>(s), reinterpret_cast<CUdeviceptr>(flag), token, 0) != CUDA_SUCCESS)
          return record_cuda_error(cudaErrorUnknown);
      }
  if ((e = cudaEventRecord(g_events.ev[1], sp)) != cudaSuccess) return record_cuda_error(e);
  if (rings == 2 && (e = cudaEventRecord(g_events.ev[2], ring_stream[1])) != cudaSuccess) return record_cuda_error(e);
  if ((e = cudaStreamWaitEvent(sc, g_events.ev[1], 0)) != cudaSuccess) return record_cuda_error(e);
  if (rings == 2 && (e = cudaStreamWaitEvent(sc, g_events.ev[2], 0)) != cudaSuccess) return record_cuda_error(e);
  return COMPASS_OK;
}

static int decomp_call(const compass_problem* pr, const void* const* A, const void* const* B, void* const* out, void* ws,
                       size_t ws_bytes, void* stream_compute, void* stream_copy, bool comm_only) {
  int st = validate_problem(pr, -1, true);
  if (st != COMPASS_OK) return st;
  if (pr->d > 16) return COMPASS_ERR_UNSUPPORTED;
  st = validate_pointers(A, B, out, pr->P);
  if (st != COMPASS_OK) return st;
  st = validate_workspace(pr, COMPASS_WS_DECOMP, ws, ws_bytes);
  if (st != COMPASS_OK) return st;
  std::lock_guard<std::mutex> lock(g_events.mu);
  st = g_events.ensure(pr->d + 1);
  if (st != COMPASS_OK) return st;
  cudaStream_t sc = static_cast<cudaStream_t>(stream_compute), sp = static_cast<cudaStream_t>(stream_copy);
  if (pr->op == COMPASS_OP_AG_GEMM) return decomp_ag(pr, A, B, out, static_cast<uint8_t*>(ws), sc, sp, g_events.ev, comm_only);
  return decomp_rs(pr, A, B, out, static_cast<uint8_t*>(ws), sc, sp, g_events.ev, comm_only);
}

extern "C" int compass_decomp(const compass_problem* pr, const void* const* A, const void* const* B, void* const* out,
                              void* ws, size_t ws_bytes, void* stream_compute, void* stream_copy) {
  return decomp_call(pr, A, B, out, ws, ws_bytes, stream_compute, stream_copy, false);
}

extern "C" int compass_decomp_comm(const compass_problem* pr, const void* const* A, const void* const* B, void* const* out,
                                   void* ws, size_t ws_bytes, void* stream_compute, void* stream_copy) {
  return decomp_call(pr, A, B, out, ws, ws_bytes, stream_compute, stream_copy, true);
}

extern "C" int compass_fused_host(const compass_problem* pr, const void* const* A_host, const void* const* B_host,
                                  void* const* out_host, void* staging, size_t staging_bytes, size_t* needed, void* ws,
                                  size_t ws_bytes, void* stream) {
  int st = validate_problem(pr, -1, false);
  if (st != COMPASS_OK) return st;
  const int P = pr->P;
  const bool ag = pr->op == COMPASS_OP_AG_GEMM;
  const size_t a_bytes = size_t(ag ? pr->M / P : pr->M) * size_t(pr->K) * 2;
  const size_t b_bytes = size_t(pr->N) * size_t(pr->K) * 2;
  const size_t o_bytes = size_t(ag ? pr->M : pr->M / P) * size_t(pr->N) * 2;
  const size_t total = size_t(P) * (align_up(a_bytes) + align_up(b_bytes) + align_up(o_bytes));
  if (needed) *needed = total;
  if (staging == nullptr) return needed ? COMPASS_OK : COMPASS_ERR_INVALID_ARG;
  if (staging_bytes < total) return COMPASS_ERR_BUFFER_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(staging) & (kAlign - 1)) != 0) return COMPASS_ERR_ALIGNMENT;
  if (A_host == nullptr || B_host == nullptr || out_host == nullptr) return COMPASS_ERR_INVALID_ARG;
  for (int r = 0; r < P; ++r)
    if (!A_host[r] || !B_host[r] || !out_host[r]) return COMPASS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(staging);
  const void* dA[kMaxP];
  const void* dB[kMaxP];
  void* dO[kMaxP];
  for (int r = 0; r < P; ++r) {
    dA[r] = base + size_t(r) * align_up(a_bytes);
    dB[r] = base + size_t(P) * align_up(a_bytes) + size_t(r) * align_up(b_bytes);
    dO[r] = base + size_t(P) * (align_up(a_bytes) + align_up(b_bytes)) + size_t(r) * align_up(o_bytes);
  }
  cudaError_t e;
  for (int r = 0; r < P; ++r) {
    if ((e = cudaMemcpyAsync(const_cast<void*>(dA[r]), A_host[r], a_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess)
      return record_cuda_error(e);
    if ((e = cudaMemcpyAsync(const_cast<void*>(dB[r]), B_host[r], b_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess)
      return record_cuda_error(e);
  }
  st = fused_call(pr, pr->op, dA, dB, dO, ws, ws_bytes, stream);
  if (st != COMPASS_OK) return st;
  for (int r = 0; r < P; ++r)
    if ((e = cudaMemcpyAsync(out_host[r], dO[r], o_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
      return record_cuda_error(e);
  return COMPASS_OK;
}

extern "C" const char* compass_status_string(int status) {
  switch (status) {
    case COMPASS_OK: return "ok";
    case COMPASS_ERR_INVALID_ARG: return "invalid argument";
    case COMPASS_ERR_SHAPE: return "shape not divisible as required";
    case COMPASS_ERR_UNSUPPORTED: return "unsupported dtype or size";
    case COMPASS_ERR_ALIGNMENT: return "pointer or row pitch not 16-byte aligned";
    case COMPASS_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case COMPASS_ERR_CUDA: return "CUDA call failed";
    case COMPASS_ERR_TIMEOUT: return "device-side wait timed out";
    case COMPASS_ERR_SCRATCH_LIMIT: return "problem exceeds the built-in scratch array of the no-allocation entry point";
    default: return "unknown status";
  }
}

extern "C" int compass_set_wait_limit_us(uint32_t microseconds) {
  g_wait_limit_us.store(microseconds, std::memory_order_relaxed);
  return COMPASS_OK;
}
extern "C" int compass_tensor_map_cache_stats(uint64_t* hits, uint64_t* misses) {
  if (hits == nullptr || misses == nullptr) return COMPASS_ERR_INVALID_ARG;
  tensor_map_cache_stats(hits, misses);
  return COMPASS_OK;
}
extern "C" int compass_test_drop_flag_writes(int count) {
  if (count < 0) return COMPASS_ERR_INVALID_ARG;
  g_drop_flag_writes.store(count);
  return COMPASS_OK;
}
extern "C" int compass_last_cuda_error(void) { return g_last_cuda_error.load(); }
extern "C" uint64_t compass_kernel_launch_count(void) { return g_kernel_launches.load(); }
