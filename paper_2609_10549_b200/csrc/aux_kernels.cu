// HBM-bound helper kernels of the InterDecom path (Section II-B): the
// sub-ReduceScatter that sums the P ranks' BF16 partial rows of one row slice
// into the owners' output rows (FP32 accumulation, ranks in ascending order,
// one BF16 rounding).
#include "internal.h"
#include "ptx_sm100.cuh"

namespace compass {

namespace {

struct ReduceParams {
  const uint4* partial[kMaxP];   // [M x N] BF16 each
  uint4* out[kMaxP];             // [m x N] BF16 each
  int32_t P;
  int64_t m;                     // rows per owner
  int64_t n_vec;                 // N / 8 (16-byte vectors per row)
  int64_t slice_begin;           // first row of the slice inside every owner's block
  int64_t slice_rows;
};

__device__ __forceinline__ void accumulate_bf16x8(float (&acc)[8], const uint4& v) {
  acc[0] += __uint_as_float(v.x << 16);
  acc[1] += __uint_as_float(v.x & 0xFFFF0000u);
  acc[2] += __uint_as_float(v.y << 16);
  acc[3] += __uint_as_float(v.y & 0xFFFF0000u);
  acc[4] += __uint_as_float(v.z << 16);
  acc[5] += __uint_as_float(v.z & 0xFFFF0000u);
  acc[6] += __uint_as_float(v.w << 16);
  acc[7] += __uint_as_float(v.w & 0xFFFF0000u);
}

__global__ void __launch_bounds__(256) reduce_partials_kernel(const __grid_constant__ ReduceParams p) {
  const int64_t per_owner = p.slice_rows * p.n_vec;
  const int64_t total = per_owner * p.P;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += int64_t(gridDim.x) * blockDim.x) {
    const int c = int(i / per_owner);
    const int64_t w = i - int64_t(c) * per_owner;
    const int64_t row = w / p.n_vec;
    const int64_t col = w - row * p.n_vec;
    const int64_t src = (int64_t(c) * p.m + p.slice_begin + row) * p.n_vec + col;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    // four ranks' vectors are fetched before the first is added, so that a thread keeps 64 bytes in flight
    int q = 0;
    for (; q + 4 <= p.P; q += 4) {
      const uint4 v0 = __ldg(p.partial[q] + src);
      const uint4 v1 = __ldg(p.partial[q + 1] + src);
      const uint4 v2 = __ldg(p.partial[q + 2] + src);
      const uint4 v3 = __ldg(p.partial[q + 3] + src);
      accumulate_bf16x8(acc, v0);
      accumulate_bf16x8(acc, v1);
      accumulate_bf16x8(acc, v2);
      accumulate_bf16x8(acc, v3);
    }
#pragma unroll 1
    for (; q < p.P; ++q) {
      const uint4 v = __ldg(p.partial[q] + src);
      accumulate_bf16x8(acc, v);
    }
    uint4 r;
    r.x = ptx::pack_bf16x2(acc[0], acc[1]);
    r.y = ptx::pack_bf16x2(acc[2], acc[3]);
    r.z = ptx::pack_bf16x2(acc[4], acc[5]);
    r.w = ptx::pack_bf16x2(acc[6], acc[7]);
    p.out[c][(p.slice_begin + row) * p.n_vec + col] = r;
  }
}

// Sub-AllGather of one InterDecom stage as ONE launch (what a library collective would be): row
// slice [slice_begin, +slice_rows) of every shard goes to every rank's gather buffer.  Every
// 16-byte vector is read once and written to the P destinations.
struct GatherParams {
  const uint4* shard[kMaxP];     // A_q [m x K]
  uint4* gather[kMaxP];          // G_r [M x K]
  int32_t P;
  int64_t m;
  int64_t k_vec;                 // K / 8
  int64_t slice_begin, slice_rows;
};

__global__ void __launch_bounds__(256) gather_slices_kernel(const __grid_constant__ GatherParams p) {
  const int64_t per_shard = p.slice_rows * p.k_vec;
  const int64_t total = per_shard * p.P;
  const int64_t stride = int64_t(gridDim.x) * blockDim.x;
  // Four vectors per thread are fetched before the first is stored (64 bytes of reads in flight per thread); every
  // vector then goes to the P gather buffers with streaming stores: the copies are not read again by this kernel and
  // should not push the GEMM's operands out of L2.
  constexpr int kUnroll = 4;
  for (int64_t i0 = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i0 < total; i0 += stride * kUnroll) {
    uint4 v[kUnroll];
    int64_t dst[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t i = i0 + u * stride;
      dst[u] = -1;
      if (i < total) {
        const int q = int(i / per_shard);
        const int64_t w = i - int64_t(q) * per_shard;
        v[u] = __ldg(p.shard[q] + p.slice_begin * p.k_vec + w);
        dst[u] = (int64_t(q) * p.m + p.slice_begin) * p.k_vec + w;
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (dst[u] >= 0)
        for (int r = 0; r < p.P; ++r) __stcs(p.gather[r] + dst[u], v[u]);
  }
}

}  // namespace

int launch_gather_slices(const void* const* shard, void* const* gather, int P, int64_t m, int64_t K, int64_t slice_begin,
                         int64_t slice_rows, cudaStream_t stream) {
  GatherParams p;
  for (int q = 0; q < P; ++q) {
    p.shard[q] = static_cast<const uint4*>(shard[q]);
    p.gather[q] = static_cast<uint4*>(gather[q]);
  }
  p.P = P;
  p.m = m;
  p.k_vec = K / 8;
  p.slice_begin = slice_begin;
  p.slice_rows = slice_rows;
  const int64_t total = slice_rows * p.k_vec * P;
  if (total <= 0) return COMPASS_OK;
  int dev = 0, num_sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  const int64_t want = (total + 255) / 256, cap = int64_t(num_sms) * 4;
  gather_slices_kernel<<<int(want < cap ? want : cap), 256, 0, stream>>>(p);
  count_kernel_launch();
  e = cudaGetLastError();
  if (e != cudaSuccess) return record_cuda_error(e);
  return COMPASS_OK;
}

int launch_reduce_partials(const void* const* partial, int P, void* const* out, int64_t m, int64_t N, int64_t slice_begin,
                           int64_t slice_rows, cudaStream_t stream) {
  ReduceParams p;
  for (int q = 0; q < P; ++q) {
    p.partial[q] = static_cast<const uint4*>(partial[q]);
    p.out[q] = static_cast<uint4*>(out[q]);
  }
  p.P = P;
  p.m = m;
  p.n_vec = N / 8;
  p.slice_begin = slice_begin;
  p.slice_rows = slice_rows;
  const int64_t total = slice_rows * p.n_vec * P;
  if (total <= 0) return COMPASS_OK;
  int dev = 0, num_sms = 0;      // asked per call: the current device may differ from the last call's
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  int64_t want = (total + 255) / 256;
  int64_t cap = int64_t(num_sms) * 8;
  int grid = int(want < cap ? want : cap);
  reduce_partials_kernel<<<grid, 256, 0, stream>>>(p);
  count_kernel_launch();
  e = cudaGetLastError();
  if (e != cudaSuccess) return record_cuda_error(e);
  return COMPASS_OK;
}

}  // namespace compass
