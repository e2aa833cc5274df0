// Plain CUDA-core kernels: obviously-correct versions of the GEMMs and of the attention.  They are a
// debugging aid selected by PERCACHE_FLAG_REFERENCE_KERNELS (and by percache_debug_gemm); the product
// path uses the tcgen05 kernels.  Their epilogues are the same device functions the tcgen05 GEMM uses.
#include "epilogue.cuh"
#include "kernels.h"

namespace pc {

// C[M][N] = A[M][K] * B[N][K]^T, fp16 inputs, fp32 accumulate.  64x64 tile, 4x4 outputs per thread.
__global__ void __launch_bounds__(256) ref_gemm_kernel(const __half* __restrict__ A, const __half* __restrict__ B,
                                                       float* __restrict__ C, int M, int N, int K) {
  __shared__ float As[16][64 + 1];
  __shared__ float Bs[16][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int i = threadIdx.x; i < 64 * 16; i += 256) {
      const int r = i >> 4, kk = i & 15;
      const int gm = m0 + r, gn = n0 + r;
      As[kk][r] = (gm < M && k0 + kk < K) ? __half2float(A[static_cast<size_t>(gm) * K + k0 + kk]) : 0.f;
      Bs[kk][r] = (gn < N && k0 + kk < K) ? __half2float(B[static_cast<size_t>(gn) * K + k0 + kk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) acc[i][jj] = fmaf(a[i], b[jj], acc[i][jj]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int gn = n0 + tx * 4 + jj;
      if (gn < N) C[static_cast<size_t>(gm) * N + gn] = acc[i][jj];
    }
  }
}
void launch_ref_gemm(const __half* A, const __half* B, float* C, int M, int N, int K, cudaStream_t s) {
  if (M <= 0) return;
  dim3 grid((N + 63) / 64, (M + 63) / 64);
  ref_gemm_kernel<<<grid, 256, 0, s>>>(A, B, C, M, N, K);
}

__global__ void ref_qkv_epilogue_kernel(const float* __restrict__ C, int M, QkvEpilogue e) {
  const int n_hb = e.n_q_heads + 2 * e.n_kv_heads;
  const int64_t n = static_cast<int64_t>(M) * n_hb * 16;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int seg = static_cast<int>(i % 16);
  const int hb = static_cast<int>((i / 16) % n_hb);
  const int row = static_cast<int>(i / (16 * n_hb));
  const float* src = C + static_cast<size_t>(row) * (n_hb * HEAD_DIM) + hb * HEAD_DIM + seg * 4;
  qkv_store4(e, row, load_qkv_row(e, row), hb, seg * 4, make_float4(src[0], src[1], src[2], src[3]),
             make_float4(src[ROPE_HALF], src[ROPE_HALF + 1], src[ROPE_HALF + 2], src[ROPE_HALF + 3]));
}
void launch_ref_qkv_epilogue(const float* C, int M, const QkvEpilogue& e, cudaStream_t s) {
  if (M <= 0) return;
  const int64_t n = static_cast<int64_t>(M) * (e.n_q_heads + 2 * e.n_kv_heads) * 16;
  ref_qkv_epilogue_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(C, M, e);
}

__global__ void ref_residual_epilogue_kernel(const float* __restrict__ C, int M, int N, ResidualEpilogue e) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= static_cast<int64_t>(M) * (N / 4)) return;
  const int row = static_cast<int>(i / (N / 4)), col = static_cast<int>(i % (N / 4)) * 4;
  const float* c = C + static_cast<size_t>(row) * N + col;
  residual_add4(e, row, col, make_float4(c[0], c[1], c[2], c[3]));
}
void launch_ref_residual_epilogue(const float* C, int M, int N, const ResidualEpilogue& e, cudaStream_t s) {
  if (M <= 0) return;
  const int64_t n = static_cast<int64_t>(M) * (N / 4);
  ref_residual_epilogue_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(C, M, N, e);
}

// C is [M][2F] with gate/up interleaved in blocks of `blk` columns: [gate blk | up blk | gate blk | ...]
__global__ void ref_swiglu_epilogue_kernel(const float* __restrict__ C, int M, int F, int blk, SwigluEpilogue e) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= static_cast<int64_t>(M) * (F / 4)) return;
  const int row = static_cast<int>(i / (F / 4)), j0 = static_cast<int>(i % (F / 4)) * 4;
  const int b = j0 / blk, jj = j0 % blk;
  const float* g = C + static_cast<size_t>(row) * (2 * F) + static_cast<size_t>(2 * b) * blk + jj;
  swiglu_store4(e, row, j0, make_float4(g[0], g[1], g[2], g[3]),
                make_float4(g[blk], g[blk + 1], g[blk + 2], g[blk + 3]));
}
void launch_ref_swiglu_epilogue(const float* C, int M, int F, int blk, const SwigluEpilogue& e, cudaStream_t s) {
  if (M <= 0) return;
  const int64_t n = static_cast<int64_t>(M) * (F / 4);
  ref_swiglu_epilogue_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(C, M, F, blk, e);
}

// Causal GQA attention, one block of 128 threads per (new row, query head).  Keys are taken in
// chunks of 512: scores into shared memory (thread = key), running max / sum, then thread = output
// column accumulates P·V for the chunk.
constexpr int REF_ATT_CHUNK = 512;
__global__ void __launch_bounds__(128)
ref_attention_kernel(const __half* __restrict__ q, const __half* __restrict__ kctx, const __half* __restrict__ vctx,
                     __half* __restrict__ out, const int32_t* __restrict__ row_pos,
                     const int32_t* __restrict__ row_ctx0, int n_q_heads, int n_kv_heads) {
  __shared__ float qs[HEAD_DIM];
  __shared__ float sc[REF_ATT_CHUNK];
  __shared__ float red[4];
  const int row = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  const int g = h / (n_q_heads / n_kv_heads);
  const int kv_dim = n_kv_heads * HEAD_DIM;
  const int n_keys = row_pos[row] + 1;
  const size_t ctx0 = static_cast<size_t>(row_ctx0[row]);
  qs[tid] = __half2float(q[(static_cast<size_t>(row) * n_q_heads + h) * HEAD_DIM + tid]);
  __syncthreads();
  const float scale = 0.08838834764831845f;   // 1/sqrt(128)
  float m_run = -INFINITY, l_run = 0.f, acc = 0.f;
  for (int k0 = 0; k0 < n_keys; k0 += REF_ATT_CHUNK) {
    const int nk = min(REF_ATT_CHUNK, n_keys - k0);
    float lmax = -INFINITY;
    for (int t = tid; t < nk; t += 128) {
      const __half2* kr = reinterpret_cast<const __half2*>(kctx + (ctx0 + k0 + t) * kv_dim + g * HEAD_DIM);
      float s = 0.f;
#pragma unroll 8
      for (int e = 0; e < HEAD_DIM / 2; ++e) {
        const float2 kk = __half22float2(kr[e]);
        s = fmaf(qs[2 * e], kk.x, s);
        s = fmaf(qs[2 * e + 1], kk.y, s);
      }
      s *= scale;
      sc[t] = s;
      lmax = fmaxf(lmax, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lmax = fmaxf(lmax, __shfl_xor_sync(0xffffffffu, lmax, o));
    if ((tid & 31) == 0) red[tid >> 5] = lmax;
    __syncthreads();
    const float cmax = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    const float m_new = fmaxf(m_run, cmax);
    const float corr = __expf(m_run - m_new);       // 0 on the first chunk (m_run = -inf)
    __syncthreads();
    float lsum = 0.f;
    for (int t = tid; t < nk; t += 128) {
      const float p = __expf(sc[t] - m_new);
      sc[t] = p;
      lsum += p;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
    if ((tid & 31) == 0) red[tid >> 5] = lsum;
    __syncthreads();
    l_run = l_run * corr + (red[0] + red[1] + red[2] + red[3]);
    acc *= corr;
    for (int t = 0; t < nk; ++t)
      acc = fmaf(sc[t], __half2float(vctx[(ctx0 + k0 + t) * kv_dim + g * HEAD_DIM + tid]), acc);
    m_run = m_new;
    __syncthreads();
  }
  out[(static_cast<size_t>(row) * n_q_heads + h) * HEAD_DIM + tid] = to_half_sat(acc / l_run);
}
void launch_ref_attention(const __half* q, const __half* kctx, const __half* vctx, __half* out, const int32_t* row_pos,
                          const int32_t* row_ctx0, int M, int n_q_heads, int n_kv_heads, cudaStream_t s) {
  if (M <= 0) return;
  dim3 grid(M, n_q_heads);
  ref_attention_kernel<<<grid, 128, 0, s>>>(q, kctx, vctx, out, row_pos, row_ctx0, n_q_heads, n_kv_heads);
}

}  // namespace pc
