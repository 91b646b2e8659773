/*
 * compass.h -- C ABI of the B200 (sm_100a) implementation of Compass's
 * tensor-parallel hot path: fused AllGather+GEMM and GEMM+ReduceScatter whose
 * tiles are visited in the order of the double-ring chunk schedule
 * (TA-IntraFusion, Section III), the decomposed pipeline (ODP-InterDecom,
 * Section IV) and the strategy selector (Algorithm 1, Section V).
 *
 * The tensor-parallel group is P logical ranks on ONE GPU: every rank's
 * shards and outputs are separate device allocations, passed as arrays of P
 * pointers.  All tensors are BF16, row-major, densely packed:
 *
 *   AllGather+GEMM   (Section II-A): rank r holds A_r [M/P x K] and the
 *       weight shard B_r stored K-major as [N x K] (N = columns PER RANK);
 *       the call produces C_r [M x N] = [A_0; ...; A_{P-1}] * B_r^T for all r.
 *   GEMM+ReduceScatter (Section II-A): rank r holds A_r [M x K] (K = PER-RANK
 *       slice of the contraction) and B_r [N x K]; the call produces
 *       Out_r [M/P x N] = rows [r*M/P, (r+1)*M/P) of sum_q A_q * B_q^T.
 *
 * Accumulation is FP32, outputs are rounded once to BF16 (round to nearest
 * even) unless a variant says otherwise.
 *
 * Ownership and errors.  The caller owns every buffer, including the
 * workspace; the library allocates no device memory.  Pointer arrays live in
 * host memory and are read before the call returns; the tensors they point to
 * are device memory unless an entry point says "host".  Device work is
 * asynchronous on the caller's stream(s).  Inputs are never written.  Every
 * function returns a compass_status; nothing throws, aborts or traps.
 * Arguments are checked on the host before any launch.  Device-side waits are
 * bounded: a wait that gives up records COMPASS_ERR_TIMEOUT in the status
 * block at the start of the workspace (see compass_read_status).
 *
 * CUDA graphs.  compass_ag_gemm, compass_gemm_rs, compass_decomp,
 * compass_ag_gemm_push and compass_mlp_block only enqueue kernels, copies,
 * stream memory operations and event record/wait pairs that fork from and
 * join back into the compute stream, so they can be called while that stream
 * is being captured; a replay works on the current contents of
 * the buffers whose addresses were captured.  The first call on a device
 * should come before any capture (it sets kernel attributes and creates the
 * library's events).
 */
#ifndef COMPASS_H
#define COMPASS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define COMPASS_MAX_P 16            /* largest tensor-parallel size accepted */
#define COMPASS_STATUS_BYTES 256    /* status block at the start of every workspace */
/* size of the built-in device array behind compass_gemm_rs_sequential_noalloc (32 MiB) */
#define COMPASS_NOALLOC_SCRATCH_BYTES (32u * 1024u * 1024u)

typedef enum compass_status {
  COMPASS_OK = 0,
  COMPASS_ERR_INVALID_ARG = 1,      /* NULL pointer, P < 1, rings not 1|2, d < 1, unknown op/variant */
  COMPASS_ERR_SHAPE = 2,            /* M % P, (M/P) % rings, (M/P) % d non-zero; M, N or K <= 0 */
  COMPASS_ERR_UNSUPPORTED = 3,      /* dtype other than BF16, P > COMPASS_MAX_P, sizes beyond int32 rows */
  COMPASS_ERR_ALIGNMENT = 4,        /* a tensor pointer not 16-byte aligned, or K % 8 / N % 8 non-zero
                                       (rows must be a multiple of 16 bytes for the tensor-map loads) */
  COMPASS_ERR_BUFFER_TOO_SMALL = 5, /* schedule capacity or workspace bytes */
  COMPASS_ERR_CUDA = 6,             /* a CUDA call failed; see compass_last_cuda_error() */
  COMPASS_ERR_TIMEOUT = 7,          /* a bounded device-side wait gave up (from compass_read_status) */
  COMPASS_ERR_SCRATCH_LIMIT = 8     /* the problem needs more scratch than the built-in array of the
                                       no-allocation entry point holds */
} compass_status;

enum { COMPASS_OP_AG_GEMM = 0, COMPASS_OP_GEMM_RS = 1 };
enum { COMPASS_DTYPE_BF16 = 0 };
/* GEMM+ReduceScatter variants.
 *   SEGMENTED_K: an output tile's accumulator runs over the P ranks' K-slices
 *     in ring order (the reduction tree is the tensor-core accumulator); one
 *     BF16 rounding.
 *   RING_RMW: every rank's partial tile is produced separately in that rank's
 *     schedule order and added to the partition's running sum in ring order by
 *     the GEMM epilogue.  The running sum is BF16 (what a BF16 ring transfer
 *     would carry) and travels from contributor to contributor through scratch
 *     in the workspace; the owner's contribution, scheduled last, writes the
 *     output rows (which never hold a partial sum).  The result is rounded once
 *     per contributor: it equals, on more than 99 % of
 *     the elements bit for bit, the ring reduce-scatter computed hop by hop
 *     with BF16 messages in the table's order.  Against the exact sum the
 *     error grows like sqrt(P) roundings: RMS within sqrt(P) * 2^-9, and the
 *     bound 1e-2 * max|result| + 1e-3 is met by all but about one element in
 *     1e7..1e8 at P = 8 (a few in 1e6 at P = 16), which exceed it by a few per
 *     cent.  Where that bound must hold on every element use SEGMENTED_K or
 *     RING_RMW_F32.  Needs, in the workspace, one int32 counter per 128 x 256
 *     fragment of the output (zero before the first call; every call leaves
 *     them zero, unless it reported COMPASS_ERR_TIMEOUT: then re-initialise the
 *     workspace) and 64 KB of scratch per counter (about P * (M/P) * N * 2
 *     bytes; never initialised, never read by the caller). */
/*   RING_RMW_F32: the same ordered ring accumulation with the running sum kept
 *     in FP32 (what an FP32 ring transfer would carry: twice the bytes per
 *     hop): contributors add their FP32 partial tile to it in ring order and
 *     the owner's contribution, last, writes the BF16 result -- one rounding,
 *     whatever P.  Needs the tile counters of RING_RMW and 128 KB of scratch
 *     per counter (about P * (M/P) * N * 4 bytes). */
enum { COMPASS_RS_SEGMENTED_K = 0, COMPASS_RS_RING_RMW = 1, COMPASS_RS_RING_RMW_F32 = 2 };
enum { COMPASS_STRATEGY_INTRAFUSION = 0, COMPASS_STRATEGY_INTERDECOM = 1 };
/* Launch order of the fused kernels.  Every rank's tiles are always issued in
 * that rank's schedule order (step ascending, ring 0 before ring 1).  What the
 * emulation is free to choose is how the P ranks' sequences are merged on the
 * one GPU:
 *   RANK_MAJOR: rank 0's whole sequence, then rank 1's, ... (a rank's weight
 *     shard stays in L2 while it is used; default);
 *   STEP_MAJOR: all ranks advance in lockstep: step 0 of every rank, then
 *     step 1, ... (what P GPUs running concurrently would do).
 * The ring read-modify-write variants always use STEP_MAJOR (its ordered adds
 * need contributor s of a partition to precede contributor s+1 in the launch);
 * the segmented-K variant has one block per partition and ignores the field. */
enum { COMPASS_ORDER_RANK_MAJOR = 0, COMPASS_ORDER_STEP_MAJOR = 1 };
/* Sub-AllGather of compass_decomp: one gather kernel per stage (a single launch, as a library
 * collective would be; it shares the SMs with the sub-GEMM it overlaps), or P*P device-to-device
 * copies per stage on the copy engines (no SM use, but P*P*d calls on the host). */
enum { COMPASS_COPY_KERNEL = 0, COMPASS_COPY_ENGINES = 1 };
/* Storage of the weight tensors B_r.  NK: [N][K], K contiguous (a linear layer's weight as the forward pass
 * multiplies by it) -- the default.  KN: [K][N], N contiguous: the same stored weight used by the backward pass,
 * where the data gradient multiplies by the transpose, so that AllGather+GEMM and GEMM+ReduceScatter of the
 * backward pass run on the weights as they are, without a transposed copy. */
enum { COMPASS_B_NK = 0, COMPASS_B_KN = 1 };
/* selectors for compass_workspace_bytes */
enum { COMPASS_WS_FUSED = 0, COMPASS_WS_DECOMP = 1, COMPASS_WS_PUSH = 2 };

/* Workload descriptor W = (pattern, M, N, K, world size[, d]) of Table IV and
 * Algorithm 1.  See the header comment for the meaning of M, N, K per op. */
typedef struct compass_problem {
  int32_t op;          /* COMPASS_OP_* */
  int32_t P;           /* tensor-parallel size, 1..COMPASS_MAX_P */
  int32_t rings;       /* 2 = double ring (default of the paper inside a NUMA domain), 1 = single ring */
  int32_t d;           /* decomposition degree for compass_decomp (>= 1); ignored elsewhere */
  int64_t M, N, K;
  int32_t dtype;       /* COMPASS_DTYPE_BF16 */
  int32_t rs_variant;  /* COMPASS_RS_* (GEMM+ReduceScatter only) */
  int32_t order;       /* COMPASS_ORDER_* : how the P logical ranks share the one GPU */
  int32_t copy_mode;   /* COMPASS_COPY_* : how compass_decomp moves the AllGather slices */
  int32_t b_layout;    /* COMPASS_B_* : storage of every B_r */
  int32_t ring_group;  /* COMPASS_RS_RING_RMW / _F32 only, else 0.  0 or 1: every contributor adds its own partial
                        * to the running sum (what a ring between P GPUs does).  G >= 2, a divisor of P: G consecutive
                        * contributors of a partition, in ring order, are accumulated in one tile's FP32 accumulator
                        * first (a ring between P/G nodes of G GPUs each, the node reducing internally): P/G
                        * read-modify-write passes and P/G roundings instead of P.  G = P is one pass. */
} compass_problem;

/* One line of the ring chunk schedule (Section III-B).  `part` = rings*chunk +
 * ring; with two rings ring 0 is the backward ring (r -> r-1, even partitions,
 * first half of a chunk's rows) and ring 1 the forward ring (r -> r+1, odd
 * partitions, second half); a single ring is the forward ring.  `peer` is the
 * neighbour the partition arrives from (AllGather) or is sent to
 * (ReduceScatter) and equals `rank` for the local entry.  row_begin/row_count
 * address rows of the gathered (AG) or fully reduced (RS) tensor. */
typedef struct compass_sched_entry {
  int32_t rank, step, ring, part, chunk, peer, row_begin, row_count;
} compass_sched_entry;

/* Calibrated parameters (Section IV-C, V-B; Algorithm 1 phase 2) for ONE
 * pattern: T_comp = comp_a + comp_b*FLOPs, T_comm = comm_a + comm_b*bytes with
 * FLOPs = 2*P*M*N*K and bytes = 2*P*M*K (AG) or 2*P*M*N (RS); eta(d) =
 * alpha_decomp + beta_decomp*d (Eq. 3); fusion overhead per synchronisation
 * point alpha_fusion + beta_fusion*m (Eq. 8).  Times in any one unit. */
typedef struct compass_calib {
  double comp_a, comp_b, comm_a, comm_b;
  double alpha_decomp, beta_decomp, alpha_fusion, beta_fusion;
} compass_calib;

typedef struct compass_choice {
  int32_t strategy;    /* COMPASS_STRATEGY_* */
  int32_t d_star;      /* Eq. 4-5 */
  double t_fusion;     /* Eq. 7 */
  double t_decomp;     /* Eq. 2 at d_star */
  double t_comp, t_comm, lambda;
  double t_star;       /* min(t_fusion, t_decomp) */
} compass_choice;

/* One block of a fused launch, in launch order (a diagnostic view of how a
 * call maps the schedule onto the kernel; see compass_launch_plan). */
typedef struct compass_plan_block {
  int32_t rank, step, ring, part;      /* schedule entry this block executes (rank = -1: shared by all) */
  int32_t a_tensor, a_row_begin;       /* which A pointer is read, first row inside it */
  int32_t out_tensor, out_row_begin;   /* which output pointer is written, first row inside it */
  int32_t rows;
  int32_t first_tile, tile_count;      /* position in the launch, counted in 256x256 output tiles (128x256 for blocks of
                                          fewer than 256 rows); a 512x256 tile of the kernel counts as two */
} compass_plan_block;

/* ---- schedule (Section III-A, III-B) -------------------------------------
 * Emits the ring chunk order: for every rank, P steps x `rings` entries;
 * AllGather+GEMM processes the local chunk at step 0, GEMM+ReduceScatter at
 * step P-1.  Order: rank-major, then step, then ring.  Writes rings*P*P
 * entries to `out` (host memory) and the number to *count.  With out == NULL
 * only *count is written.  Pure host integer code, deterministic. */
int compass_schedule(int op, int P, int rings, int64_t M,
                     compass_sched_entry* out, size_t capacity, size_t* count);

/* ---- fused AllGather+GEMM (TA-IntraFusion, Section III-B) ----------------
 * ONE kernel launch computes C_r for all ranks.  A tile of C_r that belongs
 * to partition p of rank r's schedule reads its A rows directly from the
 * shard of the rank that owns p (the gather is done by address, there is no
 * gather buffer) and is issued in that rank's schedule order; the P ranks'
 * sequences are merged rank-major by default, step-major on request
 * (problem->order).
 *   A: P device pointers, A[r] = [M/P x K];  B: P device pointers [N x K];
 *   C: P device pointers [M x N] (every element is written).
 *   workspace: >= compass_workspace_bytes(problem, COMPASS_WS_FUSED) bytes of
 *   device memory, 256-byte aligned, whose status block was zeroed once with
 *   compass_workspace_init.  cuda_stream: a cudaStream_t (NULL = default). */
int compass_ag_gemm(const compass_problem* problem, const void* const* A, const void* const* B,
                    void* const* C, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- fused AllGather+GEMM driven by data readiness (Section III-B) --------
 * The paper's mechanism itself -- push-based transfers by the DMA engines plus
 * semaphores that the GEMM tiles wait on -- emulated on one GPU.  Every rank r
 * has a private gather buffer G_r [M x K] in the workspace.  On stream_copy,
 * step by step (s = 1 .. P-1) and ring by ring, the partition that rank r
 * processes at step s is pushed by a device-to-device copy from its upstream
 * neighbour (from the neighbour's shard at s = 1, from the neighbour's gather
 * buffer afterwards: hop by hop, as on the ring) into G_r, and a readiness
 * flag is raised in stream order behind the copy.  ONE GEMM kernel on
 * stream_compute runs concurrently: step-0 tiles read the local shard at once
 * and hide the first transfers; a tile of a later step is loaded only after
 * its partition's flag is up (bounded wait; a wait that gives up reports
 * COMPASS_ERR_TIMEOUT).  Tiles are issued step-major (all ranks in lockstep).
 * Arguments as compass_ag_gemm; workspace >= compass_workspace_bytes(problem,
 * COMPASS_WS_PUSH).  On return all work is ordered before later work on
 * stream_compute.  stream_copy must differ from stream_compute.  With two
 * rings the backward ring's copy chain runs on stream_copy and the forward
 * ring's on a stream of the library's own (one per device, created on first
 * use): the rings move disjoint partitions, so their chains are independent.
 * The kernel is launched before the copies are enqueued, so that it does not
 * wait for the host to issue them.
 * Precondition: the kernel's tiles wait for flags while holding their SMs, and
 * its grid is sized for an otherwise idle GPU.  Run nothing else on the GPU's
 * SMs for the duration of the call (another kernel of this process that
 * occupies SMs can keep a tile that others wait for from starting; the waits
 * then run into the limit).  Read compass_read_status after the call: on
 * COMPASS_ERR_TIMEOUT the output is incomplete. */
int compass_ag_gemm_push(const compass_problem* problem, const void* const* A, const void* const* B,
                         void* const* C, void* workspace, size_t workspace_bytes,
                         void* stream_compute, void* stream_copy);

/* ---- fused GEMM+ReduceScatter (Section III-B, last paragraph) ------------
 * ONE kernel launch, no separate reduce kernel.  For partition p = (chunk c,
 * ring g) the contributions are added in the order in which the running sum
 * would travel the ring, ending with the owner c.
 *   A: P device pointers [M x K];  B: P device pointers [N x K];
 *   Out: P device pointers [M/P x N] (every element is written).
 * Precondition of COMPASS_RS_RING_RMW and COMPASS_RS_RING_RMW_F32: contributor s of an output tile waits,
 * holding its SM, for contributor s-1, which is earlier in the launch; that
 * is deadlock-free because all CTAs of the launch are resident at once, and
 * the grid is sized for an otherwise idle GPU.  Run nothing else on the GPU's
 * SMs for the duration of the call, and read compass_read_status after it: on
 * COMPASS_ERR_TIMEOUT the output is incomplete and the tile counters are
 * dirty (re-initialise the workspace).  The segmented-K variant has no such
 * waits. */
int compass_gemm_rs(const compass_problem* problem, const void* const* A, const void* const* B,
                    void* const* Out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- ODP-InterDecom (Section II-B, IV) -----------------------------------
 * The same result as the fused calls, computed as problem->d sub-operators
 * pipelined on two streams.  The operator is split along rows: with
 * s = M/P/d, sub-operator j handles rows [j*s, (j+1)*s) of every chunk.
 *   AG: sub-collective j = row slice j of every shard copied into every
 *       rank's gather buffer (in the workspace) on stream_copy, by one gather
 *       kernel or by copy-engine copies (problem->copy_mode); sub-GEMM j on
 *       stream_compute once they have landed.
 *   RS: sub-GEMM j writes every rank's BF16 partial rows (workspace) on
 *       stream_compute; sub-collective j = a reduce kernel on stream_copy
 *       that sums the P partial slices in FP32 into the owners' rows.
 * d = 1 is sequential execution.  On return all work is ordered before later
 * work on stream_compute.  out = C (AG) or Out (RS) as in the fused calls.
 * stream_copy must differ from stream_compute for overlap (equal is legal). */
int compass_decomp(const compass_problem* problem, const void* const* A, const void* const* B,
                   void* const* out, void* workspace, size_t workspace_bytes,
                   void* stream_compute, void* stream_copy);

/* The d sub-collectives of compass_decomp alone, without the sub-GEMMs: what
 * Section IV-C calls T_comm, made measurable on its own (the sub-AllGathers
 * of AG: every shard's row slices into the P gather buffers; the
 * sub-ReduceScatters of RS: the P BF16 partial buffers of the workspace, as
 * they are -- zero after compass_workspace_init, or what the last
 * compass_decomp left there -- summed into `out`).  Same arguments, streams
 * and ordering as compass_decomp; B is not read.  These phases are bound by
 * HBM bandwidth: AG reads M*K*2 bytes and writes P times that, RS reads
 * P*M*N*2 bytes and writes M*N*2. */
int compass_decomp_comm(const compass_problem* problem, const void* const* A, const void* const* B,
                        void* const* out, void* workspace, size_t workspace_bytes,
                        void* stream_compute, void* stream_copy);

/* ---- strategy selector (Algorithm 1, Eq. 2-8) ------------------------------
 * T_comp, T_comm and lambda come from the calibrated linear models; the
 * decomposition degree d* from Eq. 4-5 (restricted to degrees that divide
 * M/P); the answer is the strategy with the smaller predicted time, T_decomp
 * (Eq. 2 at d*) or T_fusion (Eq. 7-8), IntraFusion only if strictly faster.
 * Host arithmetic only.
 * compass_select evaluates Eq. 5 with min(lambda, 1/lambda) in place of the
 * printed 1/lambda -- a deliberate departure: that is the stationary point of
 * Eq. 2 in both regimes, and it coincides with the printed form whenever
 * T_comp >= T_comm (see compass_model_optimal_degree).  compass_select_ex with
 * eq5_as_printed != 0 runs the selector on Eq. 5 exactly as printed. */
int compass_select(const compass_problem* problem, const compass_calib* calib, compass_choice* out);
int compass_select_ex(const compass_problem* problem, const compass_calib* calib, int eq5_as_printed,
                      compass_choice* out);

/* ---- the tensor-parallel MLP block (Section II-A, the two-layer MLP figure) --
 * AllGather -> GEMM0 (W0 column-parallel) -> GEMM1 (W1 row-parallel) ->
 * ReduceScatter as TWO fused kernels back to back on one stream: the fused
 * AllGather+GEMM with the element-wise function applied to the FP32
 * accumulator in its epilogue, then the fused GEMM+ReduceScatter reading the
 * BF16 result:
 *     H_r   = act( gather(X) * W0_r )
 *     Out_c = rows [c*M/P, (c+1)*M/P) of  sum_q H_q * W1_q
 * The paper's text puts nothing between the two GEMMs (COMPASS_ACT_NONE); an
 * MLP has an activation there, so two are offered:
 *   GELU_TANH: 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))
 *   SWIGLU:    the rows of W0_r alternate (gate_0, up_0, gate_1, up_1, ...), so
 *              that GEMM0's columns 2j and 2j+1 are gate_j and up_j;
 *              H[:, j] = gate_j / (1 + exp(-gate_j)) * up_j and H has ffn / 2
 *              columns (ffn must be a multiple of 16).
 *   X:   P device pointers, X[r]  = [M/P x hidden]
 *   W0:  P device pointers, W0[r] = [ffn x hidden]       (K-major, as every weight)
 *   H:   P device pointers, H[r]  = [M x hc], hc = ffn (ffn / 2 with SWIGLU);
 *        caller-owned intermediate, every element is written
 *   W1:  P device pointers, W1[r] = [hidden x hc]
 *   Out: P device pointers, Out[r] = [M/P x hidden]
 *   workspace: >= compass_mlp_workspace_bytes bytes, 256-byte aligned, zeroed
 *   once with compass_workspace_init; compass_read_status reports a bounded
 *   wait of either kernel that gave up.
 * Backward pass: the data gradients of the literal block (no activation) are
 * the same chain run on the stored weights with COMPASS_B_KN --
 * dH_r = gather(dOut) * W1_r and dX_c = rows of sum_q dH_q * W0_q, i.e. the
 * call (dOut, W1, dH, W0, dX) with hidden and ffn unchanged.  Activation
 * derivatives and weight gradients are not part of this library. */
enum { COMPASS_ACT_NONE = 0, COMPASS_ACT_GELU_TANH = 1, COMPASS_ACT_SWIGLU = 2 };
typedef struct compass_mlp {
  int32_t P;           /* tensor-parallel size */
  int32_t rings;       /* 1 or 2, as in compass_problem */
  int64_t M;           /* rows of the gathered input (all ranks) */
  int64_t hidden;      /* K of GEMM0 = N of GEMM1 */
  int64_t ffn;         /* N of GEMM0 per rank */
  int32_t activation;  /* COMPASS_ACT_* */
  int32_t rs_variant;  /* COMPASS_RS_* of the second kernel */
  int32_t order;       /* COMPASS_ORDER_* of the first kernel */
  int32_t b_layout;    /* COMPASS_B_* : storage of W0_r and W1_r (KN: [hidden x ffn] and [hc x hidden]) */
} compass_mlp;
int compass_mlp_workspace_bytes(const compass_mlp* mlp, size_t* bytes);
int compass_mlp_block(const compass_mlp* mlp, const void* const* X, const void* const* W0, void* const* H,
                      const void* const* W1, void* const* Out, void* workspace, size_t workspace_bytes,
                      void* cuda_stream);

/* ---- models, individually (host) ----------------------------------------- */
/* Eq. 2-3: (d-1)*max(T_comp,T_comm)/d*(alpha+beta*d) + T_comp/d + T_comm/d. */
int compass_model_decomp_time(double t_comp, double t_comm, double alpha, double beta, int d, double* out);
/* Eq. 4-5.  d_max: largest admissible degree (1..16).  as_printed != 0
 * evaluates Eq. 5 literally with 1/lambda; 0 uses min(lambda, 1/lambda),
 * which is the stationary point of Eq. 2 in both regimes.  *d_continuous
 * (may be NULL) receives the argument of P_2, or -1 if it does not exist. */
int compass_model_optimal_degree(double t_comp, double t_comm, double alpha, double beta, int d_max,
                                 int as_printed, int* d_final, double* d_continuous);
/* Eq. 7-8 with equal chunks: T_comp/n per chunk, T_comm/(n-1) per step. */
int compass_model_fusion_time(double t_comp, double t_comm, int n_chunks, double alpha_f, double beta_f,
                              double m_volume, double* out);
/* One-time offline regressions (Section IV-C): eta measured at each sample
 * (t_comp[i], t_comm[i], d[i] > 1, t_measured[i]) regressed on d. */
int compass_calib_fit_decomp(const double* t_comp, const double* t_comm, const int* d, const double* t_measured,
                             size_t n, double* alpha, double* beta);
/* Least-squares line y = a + b*x (the linear T_comp and T_comm models of
 * Section IV-B are fitted with it); a single distinct x gives (mean y, 0). */
int compass_calib_fit_line(const double* x, const double* y, size_t n, double* a, double* b);
/* Residual of Eq. 7 per synchronisation point regressed on the message volume m. */
int compass_calib_fit_fusion(const double* t_comp, const double* t_comm, const int* n_chunks, const double* m_volume,
                             const double* t_measured, size_t n, double* alpha_f, double* beta_f);

/* ---- helpers ------------------------------------------------------------- */
/* Workspace size in bytes for the fused call (which = COMPASS_WS_FUSED), for
 * compass_decomp (COMPASS_WS_DECOMP) or for compass_ag_gemm_push (COMPASS_WS_PUSH). */
int compass_workspace_bytes(const compass_problem* problem, int which, size_t* bytes);
/* Zero the status block and every counter of a workspace (asynchronous). */
int compass_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);
/* Synchronise the stream and return the device-side status recorded in the
 * workspace (COMPASS_OK or COMPASS_ERR_TIMEOUT); *detail (may be NULL) gets
 * a code telling which wait gave up. */
int compass_read_status(void* workspace, void* cuda_stream, int* detail);
/* Synchronise the stream and return how long CTA 0 of the last GEMM kernel
 * that used this workspace ran, in SM clock cycles and in nanoseconds (host
 * pointers, both required).  cycles / nanoseconds is the SM clock the kernel
 * really had: under the board's power cap a tensor-core kernel runs well
 * below the nominal clock, and a throughput figure can only be judged against
 * the clock it was obtained at.  A measurement aid, not part of the paper's
 * method; both values are 0 before the first launch. */
int compass_read_kernel_clock(void* workspace, void* cuda_stream, uint64_t* sm_cycles, uint64_t* nanoseconds);
/* How a launch is cut into tiles (a diagnostic view of host-side planning; no
 * GPU is touched).  decomposed = 0: the fused launch of problem->op (and
 * rs_variant, order, rings); decomposed != 0: one sub-GEMM of compass_decomp
 * with problem->d.  cta_pairs: how many clusters of two CTAs are resident at
 * once (74 on a B200; 0 = no clusters: single-CTA tiles).  Blocks of at least
 * 256 rows -- or groups of smaller blocks that share a weight tensor -- are
 * computed by CTA pairs: 512x256 tiles for the whole waves of pairs, then
 * 256x256 and 256x128 tiles for what is left, in whole rounds; the ring
 * read-modify-write variant uses 256x256 tiles only; what cannot be paired
 * runs as 128x256 tiles on single CTAs. */
typedef struct compass_tile_counts {
  int32_t cta_pairs;         /* 1: tiles computed by pairs of CTAs, 0: by single CTAs */
  int32_t blocks;            /* blocks (contiguous output row ranges) of the launch */
  int32_t rows_per_block;
  int32_t blocks_per_group;  /* consecutive blocks tiled together (1 = none) */
  int32_t tiles_512x256, tiles_256x256, tiles_256x128, tiles_128x256;
  int32_t total_tiles;
} compass_tile_counts;
int compass_tile_plan(const compass_problem* problem, int decomposed, int cta_pairs, compass_tile_counts* out);
/* The blocks of the fused launch for this problem, in launch order.  With
 * problem->ring_group = G > 1 a block stands for G consecutive contributors of a
 * partition and carries the rank and the step of the first of them; there are
 * rings * P * P / G blocks. */
int compass_launch_plan(const compass_problem* problem, compass_plan_block* out, size_t capacity, size_t* count);
/* End-to-end convenience with HOST tensors: copies A and B (host pointers,
 * pinned memory recommended) into `staging` (device, >= *staging_bytes_needed),
 * runs the fused operator of problem->op and copies the outputs back to the
 * host pointers in `out`; all asynchronous on cuda_stream.  With staging ==
 * NULL only *staging_bytes_needed is written. */
int compass_fused_host(const compass_problem* problem, const void* const* A_host, const void* const* B_host,
                       void* const* out_host, void* staging, size_t staging_bytes, size_t* staging_bytes_needed,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);
/* ---- no-allocation variant (the paper has no counterpart) -------------------
 * GEMM+ReduceScatter in its sequential form -- one GEMM that writes every
 * rank's BF16 partial product, then the reduce kernel that sums the P partials
 * in FP32 into the owners' rows (the same result, bit for bit, as
 * compass_decomp with d = 1) -- for callers that cannot hand the library a
 * workspace: a process whose device memory was all given out before this call
 * (a server or job started with a fixed memory budget that fills the GPU, a
 * plug-in inside another framework's memory pool), where a cudaMalloc for the
 * partials would fail, fragment the pool or stall every stream, or a
 * latency-critical loop that cannot afford the device-wide synchronisation of
 * cudaMalloc/cudaFree.  The caller passes only inputs and outputs:
 *   A: P device pointers [M x K];  B: P device pointers [N x K];
 *   Out: P device pointers [M/P x N] (every element is written).
 * The scratch (status block + P partial products of M*N BF16 each) is a
 * built-in device array of COMPASS_NOALLOC_SCRATCH_BYTES; every GPU on which
 * the library is loaded holds it until the process exits.  A problem with
 * 256 + P * M * N * 2 bytes (each partial rounded up to 256 bytes) beyond that
 * size is refused with COMPASS_ERR_SCRATCH_LIMIT.  The call allocates nothing:
 * no cudaMalloc, no cudaFree, no allocating library routine.
 * The first call on a device looks up the array's device address (once per
 * device, with that device current; if the CUDA runtime loads modules lazily,
 * that is also when the driver reserves the array's memory on that GPU); make
 * that first call before any stream capture begins.  All calls on a GPU share the array, which keeps what the
 * previous call left in it (the status block is cleared at the start of every
 * call; the partials are overwritten before they are read): calls ordered on
 * one stream are fine, calls that overlap on the GPU race and give undefined
 * results.  A device-side wait that gives up is recorded inside the array:
 * read it with compass_noalloc_read_status before the next no-allocation call
 * on that GPU (which clears it). */
int compass_gemm_rs_sequential_noalloc(const compass_problem* problem, const void* const* A, const void* const* B,
                                       void* const* Out, void* cuda_stream);
/* Companion of the entry point above (the paper has no counterpart): such a
 * caller never sees a workspace, so compass_read_status has nothing to read.
 * This call synchronises cuda_stream and returns the device-side status that
 * the last compass_gemm_rs_sequential_noalloc on the current device left in
 * the built-in array (COMPASS_OK or COMPASS_ERR_TIMEOUT; *detail, which may be
 * NULL, tells which wait gave up).  It allocates nothing either.  After
 * COMPASS_ERR_TIMEOUT the output rows of that call are incomplete.  Call it
 * before the next no-allocation call on that GPU, which clears the record. */
int compass_noalloc_read_status(void* cuda_stream, int* detail);

/* Bound, in microseconds, of every device-side wait of later launches (default
 * 2,000,000).  A wait that exceeds it makes the kernel record
 * COMPASS_ERR_TIMEOUT and return instead of spinning.  0 restores the default. */
int compass_set_wait_limit_us(uint32_t microseconds);
/* The library keeps the TMA tensor maps it encodes in a small per-thread
 * table keyed by (base pointer, rows, row length, box): repeated calls on the
 * same buffers skip the driver's encoding call (about a microsecond per map,
 * 2P maps per fused launch).  A map describes addresses and shapes, not
 * contents, so the table never needs invalidating; a changed pointer or shape
 * is a new key.  This call reports, over all threads since the library was
 * loaded, how many map requests were served from the table and how many were
 * encoded (host pointers, both required).  Diagnostics only. */
int compass_tensor_map_cache_stats(uint64_t* hits, uint64_t* misses);
/* Failure injection on the host, for tests of the bounded waits (the paper has
 * no counterpart): the next `count` readiness-flag writes of
 * compass_ag_gemm_push are left out -- the partition is copied but never
 * announced, as if a peer's message had been lost -- so the tile that needs it
 * gives up after the wait limit and the call's status block reads
 * COMPASS_ERR_TIMEOUT with detail 7 (the readiness-flag wait).  No GPU fault is
 * involved; the context stays usable.  0 switches the injection off. */
int compass_test_drop_flag_writes(int count);
const char* compass_status_string(int status);
int compass_last_cuda_error(void);
/* Number of kernels this library has launched since it was loaded. */
uint64_t compass_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* COMPASS_H */
