// Ring chunk schedule (Section III-A, III-B), host integer code.
//
// Forward ring: r -> r+1; backward ring: r -> r-1 (mod P).  With two rings,
// ring 0 is the backward ring and carries the even partitions (first half of
// each chunk's rows), ring 1 the forward ring with the odd partitions.  A
// partition that started at rank c has travelled s hops after s steps, so in
// AllGather+GEMM rank r processes at step s the chunk that lies s positions
// upstream of it; in GEMM+ReduceScatter a partition must finish at its owner
// after the last step, so at step s rank r works on the chunk whose owner is
// P-1-s positions downstream.
#include "internal.h"

namespace compass {

int validate_schedule_args(int op, int P, int rings, int64_t M) {
  if (op != COMPASS_OP_AG_GEMM && op != COMPASS_OP_GEMM_RS) return COMPASS_ERR_INVALID_ARG;
  if (P < 1 || (rings != 1 && rings != 2)) return COMPASS_ERR_INVALID_ARG;
  if (P > COMPASS_MAX_P) return COMPASS_ERR_UNSUPPORTED;
  if (M <= 0 || M % P != 0 || (M / P) % rings != 0) return COMPASS_ERR_SHAPE;
  if (M > INT32_MAX) return COMPASS_ERR_UNSUPPORTED;
  return COMPASS_OK;
}

static inline int wrap(int x, int P) {
  x %= P;
  return x < 0 ? x + P : x;
}

int build_schedule(int op, int P, int rings, int64_t M, compass_sched_entry* out) {
  const int32_t rows_per_chunk = int32_t(M / P);
  const int32_t rows_per_part = rows_per_chunk / rings;
  size_t n = 0;
  for (int rank = 0; rank < P; ++rank) {
    for (int step = 0; step < P; ++step) {
      for (int ring = 0; ring < rings; ++ring) {
        const int dir = (rings == 2 && ring == 0) ? -1 : +1;
        compass_sched_entry e;
        e.rank = rank;
        e.step = step;
        e.ring = ring;
        if (op == COMPASS_OP_AG_GEMM) {
          e.chunk = wrap(rank - dir * step, P);
          e.peer = (step == 0) ? rank : wrap(rank - dir, P);
        } else {
          const int hops_left = P - 1 - step;
          e.chunk = wrap(rank + dir * hops_left, P);
          e.peer = (hops_left == 0) ? rank : wrap(rank + dir, P);
        }
        e.part = rings * e.chunk + ring;
        e.row_begin = e.chunk * rows_per_chunk + ring * rows_per_part;
        e.row_count = rows_per_part;
        out[n++] = e;
      }
    }
  }
  return COMPASS_OK;
}

}  // namespace compass

extern "C" int compass_schedule(int op, int P, int rings, int64_t M, compass_sched_entry* out, size_t capacity,
                                size_t* count) {
  if (count == nullptr) return COMPASS_ERR_INVALID_ARG;
  int st = compass::validate_schedule_args(op, P, rings, M);
  if (st != COMPASS_OK) return st;
  const size_t n = size_t(rings) * size_t(P) * size_t(P);
  *count = n;
  if (out == nullptr) return COMPASS_OK;
  if (capacity < n) return COMPASS_ERR_BUFFER_TOO_SMALL;
  return compass::build_schedule(op, P, rings, M, out);
}
