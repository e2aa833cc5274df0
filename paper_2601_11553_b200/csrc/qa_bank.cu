// QA-bank lookup (paper Section 3.4.1, "Similar Query Reuse"): cosine similarity of a query embedding against
// every stored query embedding, the best entry, and the test against the threshold tau_query.
//
// HBM-bound: every launch streams the whole bank (n_entries x dim fp32) once, whatever the number of queries
// in the batch (up to QA_MAX_QUERIES, held in shared memory).  One warp per bank row: 16-byte loads, the row's
// squared norm and its dot products with all queries accumulated in the same pass.  The per-query maximum is
// kept as a 64-bit key (ordered score bits, then the complement of the index so that the lowest index wins
// ties) and merged with atomicMax.
#include <cstring>

#include "../../include/percache.h"
#include "kernels.h"
#include "ptx.cuh"

namespace pc {
namespace {

constexpr int QA_MAX_QUERIES = 8;
constexpr int QA_THREADS = 256;

// per-query maxima of the call in flight (one lookup at a time per device and process)
__device__ unsigned long long g_qa_best[QA_MAX_QUERIES];

// monotone map float -> uint32 (larger float, larger key); NaN never produced here
__device__ __forceinline__ uint32_t ordered_bits(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__host__ __device__ inline float from_ordered_bits(uint32_t k) {
  const uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  float f;
#ifdef __CUDA_ARCH__
  f = __uint_as_float(u);
#else
  memcpy(&f, &u, 4);
#endif
  return f;
}

template <int NQ>
__global__ void __launch_bounds__(QA_THREADS)
qa_top1_kernel(const float* __restrict__ bank, const float* __restrict__ queries, int n_valid, int n_entries, int dim,
               unsigned long long* __restrict__ best) {
  extern __shared__ float q_s[];                         // [NQ][dim] queries, then [NQ] inverse norms
  float* q_inv = q_s + NQ * dim;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < NQ * dim; i += QA_THREADS) q_s[i] = i < n_valid * dim ? queries[i] : 0.f;   // unused slots: zeros
  __syncthreads();
  if (warp < NQ) {
    float ss = 0.f;
    for (int i = lane; i < dim; i += 32) ss += q_s[warp * dim + i] * q_s[warp * dim + i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) q_inv[warp] = rsqrtf(fmaxf(ss, 1e-30f));
  }
  __syncthreads();
  unsigned long long local_best[NQ];
#pragma unroll
  for (int q = 0; q < NQ; ++q) local_best[q] = 0ull;
  const int n_vec = dim >> 2;
  const int warps_total = gridDim.x * (QA_THREADS / 32);
  // two bank rows per step: every query vector read from shared memory is used twice, and eight independent
  // 16-byte loads per lane are in flight
  for (int row = 2 * (blockIdx.x * (QA_THREADS / 32) + warp); row < n_entries; row += 2 * warps_total) {
    const bool two = row + 1 < n_entries;
    const float4* e0 = reinterpret_cast<const float4*>(bank + static_cast<size_t>(row) * dim);
    const float4* e1 = reinterpret_cast<const float4*>(bank + static_cast<size_t>(two ? row + 1 : row) * dim);
    float ee0 = 0.f, ee1 = 0.f, dot0[NQ], dot1[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) { dot0[q] = 0.f; dot1[q] = 0.f; }
#pragma unroll 4
    for (int v = lane; v < n_vec; v += 32) {
      const float4 x0 = __ldg(e0 + v), x1 = __ldg(e1 + v);
      ee0 += x0.x * x0.x + x0.y * x0.y + x0.z * x0.z + x0.w * x0.w;
      ee1 += x1.x * x1.x + x1.y * x1.y + x1.z * x1.z + x1.w * x1.w;
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const float4 y = *reinterpret_cast<const float4*>(q_s + q * dim + 4 * v);
        dot0[q] += x0.x * y.x + x0.y * y.y + x0.z * y.z + x0.w * y.w;
        dot1[q] += x1.x * y.x + x1.y * y.y + x1.z * y.z + x1.w * y.w;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ee0 += __shfl_xor_sync(0xffffffffu, ee0, o);
      ee1 += __shfl_xor_sync(0xffffffffu, ee1, o);
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        dot0[q] += __shfl_xor_sync(0xffffffffu, dot0[q], o);
        dot1[q] += __shfl_xor_sync(0xffffffffu, dot1[q], o);
      }
    }
    const float inv0 = rsqrtf(fmaxf(ee0, 1e-30f)), inv1 = rsqrtf(fmaxf(ee1, 1e-30f));
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
      const unsigned long long k0 = (static_cast<unsigned long long>(ordered_bits(dot0[q] * inv0 * q_inv[q])) << 32) |
                                    (0xffffffffu - static_cast<uint32_t>(row));
      local_best[q] = k0 > local_best[q] ? k0 : local_best[q];
      if (two) {
        const unsigned long long k1 = (static_cast<unsigned long long>(ordered_bits(dot1[q] * inv1 * q_inv[q])) << 32) |
                                      (0xffffffffu - static_cast<uint32_t>(row + 1));
        local_best[q] = k1 > local_best[q] ? k1 : local_best[q];
      }
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int q = 0; q < NQ; ++q)
      if (q < n_valid && local_best[q]) atomicMax(best + q, local_best[q]);
  }
}

template <int NQ>
int launch_qa(const float* bank, const float* queries, int n_valid, int n_entries, int dim, unsigned long long* best,
              int n_sms, cudaStream_t s) {
  const size_t smem = static_cast<size_t>(NQ) * (dim + 1) * sizeof(float);
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(qa_top1_kernel<NQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
    return -1;
  const int blocks = n_sms * 8;
  qa_top1_kernel<NQ><<<blocks, QA_THREADS, smem, s>>>(bank, queries, n_valid, n_entries, dim, best);
  return cudaGetLastError() == cudaSuccess ? 0 : -1;
}

}  // namespace
}  // namespace pc

using namespace pc;

extern "C" int percache_qa_top1(int32_t device, void* stream, const float* bank, int32_t n_entries, int32_t dim,
                                const float* queries, int32_t n_queries, float tau_query, int32_t* best_index,
                                float* best_score, uint8_t* hit, float* kernel_us) {
  if (!bank || !queries || !best_index || !best_score || !hit || n_entries <= 0 || dim <= 0 || dim % 4 != 0 ||
      n_queries <= 0)
    return PERCACHE_E_INVAL;
  if (n_queries > QA_MAX_QUERIES || static_cast<size_t>(QA_MAX_QUERIES) * (dim + 1) * 4 > 200 * 1024) return PERCACHE_E_CAPACITY;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int n_sms = 148;
  cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, device);
  unsigned long long* d_best = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&d_best), g_qa_best) != cudaSuccess || !d_best) {
    cudaGetLastError();
    return PERCACHE_E_CUDA;
  }
  unsigned long long h_best[QA_MAX_QUERIES];
  int rc = PERCACHE_OK;
  bool ok = cudaMemsetAsync(d_best, 0, sizeof(h_best), s) == cudaSuccess;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (kernel_us) {
    ok = ok && cudaEventCreate(&ev0) == cudaSuccess && cudaEventCreate(&ev1) == cudaSuccess;
    if (ok) cudaEventRecord(ev0, s);
  }
  // the number of query slots is a compile-time constant of the kernel (accumulators per query live in registers)
  int lrc;
  if (n_queries == 1) lrc = launch_qa<1>(bank, queries, 1, n_entries, dim, d_best, n_sms, s);
  else if (n_queries == 2) lrc = launch_qa<2>(bank, queries, 2, n_entries, dim, d_best, n_sms, s);
  else if (n_queries <= 4) lrc = launch_qa<4>(bank, queries, n_queries, n_entries, dim, d_best, n_sms, s);
  else lrc = launch_qa<8>(bank, queries, n_queries, n_entries, dim, d_best, n_sms, s);
  ok = ok && lrc == 0;
  if (kernel_us && ok) cudaEventRecord(ev1, s);
  ok = ok && cudaMemcpyAsync(h_best, d_best, sizeof(h_best), cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (!ok || cudaStreamSynchronize(s) != cudaSuccess || cudaGetLastError() != cudaSuccess) rc = PERCACHE_E_CUDA;
  if (kernel_us) {
    float ms = 0.f;
    if (rc == PERCACHE_OK && cudaEventElapsedTime(&ms, ev0, ev1) == cudaSuccess) *kernel_us = 1000.f * ms;
    if (ev0) cudaEventDestroy(ev0);
    if (ev1) cudaEventDestroy(ev1);
  }
  if (rc != PERCACHE_OK) return rc;
  for (int q = 0; q < n_queries; ++q) {
    best_index[q] = static_cast<int32_t>(0xffffffffu - static_cast<uint32_t>(h_best[q] & 0xffffffffull));
    best_score[q] = from_ordered_bits(static_cast<uint32_t>(h_best[q] >> 32));
    hit[q] = best_score[q] > tau_query ? 1 : 0;
  }
  return PERCACHE_OK;
}
