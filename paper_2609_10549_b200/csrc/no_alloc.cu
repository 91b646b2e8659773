// GEMM+ReduceScatter, sequential form (a GEMM that writes every rank's BF16
// partial product, then the reduce kernel that sums the P partials into the
// owners' rows), for callers that cannot give the library any device memory
// besides the inputs and the outputs.
//
// Who that is: code that runs inside a process whose device memory has all
// been handed out before this library is called -- an inference server or a
// training job started with a fixed memory budget that fills the GPU, or a
// plug-in living inside a host framework's memory pool -- so that a cudaMalloc
// for the P*M*N partial buffer would fail, fragment the pool or stall every
// stream while the driver serves it; and code on a latency-critical path where
// the device-wide synchronisation of cudaMalloc/cudaFree is not acceptable.
//
// The scratch (status block + partial products) therefore lives in a
// file-scope device array of fixed size.  Every GPU on which this library is
// loaded holds that array until the process exits.  All calls on one GPU share
// it: two calls that overlap on the GPU (different streams, no ordering) race
// on it and give undefined results; calls ordered on one stream are fine.
#include <mutex>

#include "internal.h"

namespace compass {
namespace {

static __device__ __align__(256) unsigned char g_noalloc_scratch[COMPASS_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mu;
unsigned char* g_noalloc_ptr[kMaxDevices] = {};

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Device address of the scratch array on the current device.  In host code the
// array's name is only a handle for the runtime; the address a kernel can use
// comes from cudaGetSymbolAddress, asked once per device with that device
// current.
int noalloc_scratch(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevices) return COMPASS_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (g_noalloc_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (ptr == nullptr) return record_cuda_error(cudaErrorInvalidSymbol);
    g_noalloc_ptr[dev] = static_cast<unsigned char*>(ptr);
  }
  *out = g_noalloc_ptr[dev];
  return COMPASS_OK;
}

}  // namespace
}  // namespace compass

using namespace compass;

extern "C" int compass_gemm_rs_sequential_noalloc(const compass_problem* pr, const void* const* A, const void* const* B,
                                                  void* const* Out, void* cuda_stream) {
  // argument checks shared with the other entry points: a workspace-size query validates the problem
  if (pr == nullptr || A == nullptr || B == nullptr || Out == nullptr) return COMPASS_ERR_INVALID_ARG;
  if (pr->op != COMPASS_OP_GEMM_RS) return COMPASS_ERR_INVALID_ARG;
  compass_problem seq = *pr;
  seq.d = 1;
  size_t need = 0;
  int st = compass_workspace_bytes(&seq, COMPASS_WS_DECOMP, &need);
  if (st != COMPASS_OK) return st;
  if (need > size_t(COMPASS_NOALLOC_SCRATCH_BYTES)) return COMPASS_ERR_SCRATCH_LIMIT;
  const int P = pr->P;
  for (int r = 0; r < P; ++r) {
    if (A[r] == nullptr || B[r] == nullptr || Out[r] == nullptr) return COMPASS_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(A[r]) | reinterpret_cast<uintptr_t>(B[r]) | reinterpret_cast<uintptr_t>(Out[r])) & 15u) != 0)
      return COMPASS_ERR_ALIGNMENT;
  }
  unsigned char* scratch = nullptr;
  st = noalloc_scratch(&scratch);
  if (st != COMPASS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  // The array keeps what the previous call left in it.  The status block must
  // start at zero; the partial products are fully overwritten before they are read.
  cudaError_t e = cudaMemsetAsync(scratch, 0, COMPASS_STATUS_BYTES, stream);
  if (e != cudaSuccess) return record_cuda_error(e);

  const int64_t m = pr->M / P;
  const size_t partial_bytes = align256(size_t(pr->M) * size_t(pr->N) * 2);
  void* W[kMaxP];
  for (int q = 0; q < P; ++q) W[q] = scratch + COMPASS_STATUS_BYTES + size_t(q) * partial_bytes;

  static thread_local GemmLaunch L;
  L.n_a = L.n_b = L.n_out = P;
  L.b_mn_major = pr->b_layout == COMPASS_B_KN;
  L.a_rows = pr->M;
  L.K = pr->K;
  L.N = pr->N;
  L.ldo = pr->N;
  L.n_seg = 1;
  L.rows_per_block = int(m);
  L.share_run = 1;
  L.epilogue = EPI_STORE;
  L.mode = GEMM_MODE_AUTO;
  L.status = reinterpret_cast<StatusBlock*>(scratch);
  L.tile_counters = nullptr;
  int n = 0;
  for (int c = 0; c < P; ++c)
    for (int q = 0; q < P; ++q) {
      L.a_ptr[q] = A[q];
      L.b_ptr[q] = B[q];
      L.out_ptr[q] = W[q];
      BlockDesc& b = L.blocks[n++];
      b = BlockDesc{};
      b.a_map = uint8_t(q);
      b.b_map = uint8_t(q);
      b.out_idx = uint8_t(q);
      b.a_row0 = int32_t(c * m);
      b.out_row0 = b.a_row0;
    }
  L.n_blocks = n;
  st = launch_gemm(L, stream);                                          // every rank's partial product
  if (st != COMPASS_OK) return st;
  return launch_reduce_partials(W, P, Out, m, pr->N, 0, m, stream);     // sum into the owners' rows
}

// The status block of the last no-allocation call on the current device, read straight from the
// built-in array (nothing is allocated: one small device-to-host copy and a stream synchronisation).
extern "C" int compass_noalloc_read_status(void* cuda_stream, int* detail) {
  unsigned char* scratch = nullptr;
  int st = noalloc_scratch(&scratch);
  if (st != COMPASS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  StatusBlock host;
  cudaError_t e = cudaMemcpyAsync(&host, scratch, sizeof(host), cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return record_cuda_error(e);
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return record_cuda_error(e);
  if (detail) *detail = host.detail;
  return host.code;
}
