// Projections for a handful of rows (decode: one row per prompt): D[M][N] = A[M][K] * W[N][K]^T with M <= 8.
//
// With so few rows the work is reading W once: a 128-row MMA tile would leave most SMs without a tile and
// the tensor core 94 % empty, so this runs on the CUDA cores and is bound by HBM.  A block first puts the M
// input rows into shared memory as fp16 (for the QKV and gate/up projections it applies the RMSNorm of the
// fp32 residual rows on the way, which saves the separate norm launch); then every warp takes pairs of W rows,
// streams them with 16-byte loads (all of a row pair's loads are in flight together), keeps 2 x M fp32 sums,
// reduces them over the warp, and lane m finishes row m with the same epilogue arithmetic as the tcgen05 GEMM:
//   QKV       rows (c, c + 64) of one head: rotation to the row's position, Q buffer / pages / context
//   residual  resid[m][n], resid[m][n + 1] += sums
//   SwiGLU    gate row and up row of column j: act[m][j] = silu(gate) * up
#include <algorithm>

#include "epilogue.cuh"
#include "kernels.h"
#include "ptx.cuh"

namespace pc {

namespace {

constexpr int SM_THREADS = 256;

struct SmallArgs {
  int32_t M, N, K;
  const float* x_f32;        // NORM input: residual rows [M][K] ...
  const float* gain;         // ... and the norm's gain [K]
  float eps;
  const __half* a_f16;       // plain input: [M][K] fp16
  const __half* w;           // [N][K] fp16
  QkvEpilogue qkv;
  ResidualEpilogue res;
  SwigluEpilogue swi;
  int32_t gu_blk;            // SwiGLU: gate / up rows are interleaved in blocks of this many rows
  int32_t k_parts;           // residual kind: pieces a row pair's K range is cut into (K / 8 / k_parts % 32 == 0)
};

__device__ __forceinline__ void half8_to_float(const uint4& v, float (&f)[8]) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// One column pair of the QKV output for one row (scalar form of qkv_store4_cs).
__device__ __forceinline__ void qkv_store1(const QkvEpilogue& e, int row, const QkvRow& rw, int hb, int c, float lo,
                                           float hi) {
  const bool is_q = hb < e.n_q_heads;
  const bool is_k = !is_q && hb < e.n_q_heads + e.n_kv_heads;
  float2 cs = make_float2(1.f, 0.f);
  if (is_q || is_k) cs = __ldg(e.rope + static_cast<size_t>(rw.pos) * ROPE_HALF + c);
  if (is_q) {
    __half* dst = e.q_out + static_cast<size_t>(row) * (e.n_q_heads * HEAD_DIM) + hb * HEAD_DIM + c;
    dst[0] = to_half_sat(lo * cs.x - hi * cs.y);
    dst[ROPE_HALF] = to_half_sat(hi * cs.x + lo * cs.y);
    return;
  }
  const int kvh = is_k ? hb - e.n_q_heads : hb - e.n_q_heads - e.n_kv_heads;
  const int kv_dim = e.n_kv_heads * HEAD_DIM;
  const __nv_bfloat16 bl = __float2bfloat16_rn(lo), bh = __float2bfloat16_rn(hi);    // the cache format
  if (rw.pool_tok >= 0) {
    __nv_bfloat16* p = (is_k ? e.kpool : e.vpool) + static_cast<size_t>(rw.pool_tok) * kv_dim + kvh * HEAD_DIM + c;
    p[0] = bl;
    p[ROPE_HALF] = bh;
  }
  if (e.skip_ctx) return;                 // a paged decode step reads the pages: nothing goes to the context
  const float l = __bfloat162float(bl), h = __bfloat162float(bh);
  __half* dst = (is_k ? e.kctx : e.vctx) + static_cast<size_t>(rw.slot) * kv_dim + kvh * HEAD_DIM + c;
  dst[0] = to_half_sat(is_k ? l * cs.x - h * cs.y : l);
  dst[ROPE_HALF] = to_half_sat(is_k ? h * cs.x + l * cs.y : h);
}

template <int KIND, int MR, bool NORM>
__global__ void __launch_bounds__(SM_THREADS) small_gemm_kernel(SmallArgs a) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __half* xs = reinterpret_cast<__half*>(smem_raw);          // [MR][K]
  __shared__ float row_scale[MR];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = a.K, M = a.M;
  pdl_launch_dependents();
  // The weights do not depend on the previous kernel: every warp asks L2 for the row pair of its first unit before
  // it waits for that kernel, so the DRAM round trip overlaps the previous kernel's tail.
  {
    const int kp = KIND == EPI_RESIDUAL ? a.k_parts : 1;
    const int wu = blockIdx.x * (SM_THREADS / 32) + warp;
    if (wu < (a.N / 2) * kp) {
      const int unit = wu / kp;
      int r0, r1;
      if (KIND == EPI_QKV) { r0 = (unit / ROPE_HALF) * HEAD_DIM + unit % ROPE_HALF; r1 = r0 + ROPE_HALF; }
      else if (KIND == EPI_SWIGLU) { r0 = (2 * (unit / a.gu_blk)) * a.gu_blk + unit % a.gu_blk; r1 = r0 + a.gu_blk; }
      else { r0 = 2 * unit; r1 = r0 + 1; }
      const int part_bytes = K * 2 / kp;
      const char* p0 = reinterpret_cast<const char*>(a.w + static_cast<size_t>(r0) * K) + (wu % kp) * part_bytes;
      const char* p1 = reinterpret_cast<const char*>(a.w + static_cast<size_t>(r1) * K) + (wu % kp) * part_bytes;
      for (int off = lane * 128; off < part_bytes; off += 32 * 128) {
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p0 + off));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p1 + off));
      }
    }
  }
  pdl_wait();

  // ---- stage the input rows (rows >= M are zero)
  if constexpr (NORM) {
    // sum of squares of every row: all threads load at once (one round trip), then warp and block reduction
    __shared__ float part_ss[SM_THREADS / 32][MR];
    float ss[MR];
#pragma unroll
    for (int m = 0; m < MR; ++m) {
      ss[m] = 0.f;
      if (m < M)
        for (int k = tid * 4; k < K; k += SM_THREADS * 4) {
          const float4 v = *reinterpret_cast<const float4*>(a.x_f32 + static_cast<size_t>(m) * K + k);
          ss[m] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
    }
#pragma unroll
    for (int m = 0; m < MR; ++m) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss[m] += __shfl_xor_sync(0xffffffffu, ss[m], o);
      if (lane == 0) part_ss[warp][m] = ss[m];
    }
    __syncthreads();
    if (tid < MR) {
      float t = 0.f;
#pragma unroll
      for (int w8 = 0; w8 < SM_THREADS / 32; ++w8) t += part_ss[w8][tid];
      row_scale[tid] = rsqrtf(t / static_cast<float>(K) + a.eps);
    }
    __syncthreads();
    for (int i = tid * 4; i < MR * K; i += SM_THREADS * 4) {
      const int m = i / K, k = i % K;
      uint2 o = make_uint2(0u, 0u);
      if (m < M) {
        const float4 v = *reinterpret_cast<const float4*>(a.x_f32 + static_cast<size_t>(m) * K + k);
        const float4 g = __ldg(reinterpret_cast<const float4*>(a.gain + k));
        const float r = row_scale[m];
        o = pack_half4(v.x * r * g.x, v.y * r * g.y, v.z * r * g.z, v.w * r * g.w);
      }
      *reinterpret_cast<uint2*>(xs + i) = o;
    }
  } else {
    for (int i = tid * 8; i < MR * K; i += SM_THREADS * 8) {
      const int m = i / K, k = i % K;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (m < M) v = *reinterpret_cast<const uint4*>(a.a_f16 + static_cast<size_t>(m) * K + k);
      *reinterpret_cast<uint4*>(xs + i) = v;
    }
  }
  __syncthreads();

  QkvRow rw{0, 0, -1};
  if (KIND == EPI_QKV && lane < M) rw = load_qkv_row(a.qkv, lane);

  // Residual kind: N is small (d_model), so a row pair's K range is cut into a.k_parts pieces for as many warps,
  // which add their partial sums atomically (as the tcgen05 residual GEMM does when it splits K).
  const int k_parts = KIND == EPI_RESIDUAL ? a.k_parts : 1;
  const int n_units = (a.N / 2) * k_parts;
  const int vecs = K / 8 / k_parts;            // 16-byte vectors of a row per part
  const int warps_total = gridDim.x * (SM_THREADS / 32);
  for (int wu = blockIdx.x * (SM_THREADS / 32) + warp; wu < n_units; wu += warps_total) {
    const int unit = wu / k_parts, v_begin = (wu % k_parts) * vecs;
    int r0, r1;
    if (KIND == EPI_QKV) {                 // columns c and c + 64 of head block hb
      r0 = (unit / ROPE_HALF) * HEAD_DIM + unit % ROPE_HALF;
      r1 = r0 + ROPE_HALF;
    } else if (KIND == EPI_SWIGLU) {       // gate and up row of output column j = unit
      r0 = (2 * (unit / a.gu_blk)) * a.gu_blk + unit % a.gu_blk;
      r1 = r0 + a.gu_blk;
    } else {
      r0 = 2 * unit;
      r1 = r0 + 1;
    }
    const uint4* w0 = reinterpret_cast<const uint4*>(a.w + static_cast<size_t>(r0) * K);
    const uint4* w1 = reinterpret_cast<const uint4*>(a.w + static_cast<size_t>(r1) * K);
    float acc0[MR], acc1[MR];
#pragma unroll
    for (int m = 0; m < MR; ++m) { acc0[m] = 0.f; acc1[m] = 0.f; }
#pragma unroll 4
    for (int v = v_begin + lane; v < v_begin + vecs; v += 32) {
      float f0[8], f1[8];
      half8_to_float(__ldg(w0 + v), f0);
      half8_to_float(__ldg(w1 + v), f1);
#pragma unroll
      for (int m = 0; m < MR; ++m) {
        float x[8];
        half8_to_float(*reinterpret_cast<const uint4*>(xs + static_cast<size_t>(m) * K + v * 8), x);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          acc0[m] = fmaf(x[e], f0[e], acc0[m]);
          acc1[m] = fmaf(x[e], f1[e], acc1[m]);
        }
      }
    }
    float s0 = 0.f, s1 = 0.f;              // lane m keeps the sums of row m
#pragma unroll
    for (int m = 0; m < MR; ++m) {
      float u0 = acc0[m], u1 = acc1[m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        u0 += __shfl_xor_sync(0xffffffffu, u0, o);
        u1 += __shfl_xor_sync(0xffffffffu, u1, o);
      }
      if (lane == m) { s0 = u0; s1 = u1; }
    }
    if (lane < M) {
      if (KIND == EPI_QKV) {
        qkv_store1(a.qkv, lane, rw, unit / ROPE_HALF, unit % ROPE_HALF, s0, s1);
      } else if (KIND == EPI_SWIGLU) {
        a.swi.act[static_cast<size_t>(lane) * a.swi.ld + unit] = to_half_sat(silu_f(s0) * s1);
      } else {
        float* p = a.res.resid + static_cast<size_t>(lane) * a.res.ld + r0;
        if (k_parts > 1) {
          atomicAdd(p, s0);
          atomicAdd(p + 1, s1);
        } else {
          float2 v = *reinterpret_cast<float2*>(p);
          v.x += s0;
          v.y += s1;
          *reinterpret_cast<float2*>(p) = v;
        }
      }
    }
  }
}

template <int KIND, bool NORM, int MR>
int launch_small_mr(const SmallArgs& a, int n_sms, cudaStream_t s) {
  const size_t smem = static_cast<size_t>(MR) * a.K * sizeof(__half);
  if (smem > 200 * 1024) return -1;
  static size_t smem_set_of[MAX_DEVICES] = {};   // per kernel instantiation and device: raised when a call needs more
  size_t& smem_set = smem_set_of[current_device_slot()];
  if (smem > smem_set) {
    if (cudaFuncSetAttribute(small_gemm_kernel<KIND, MR, NORM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess)
      return -1;
    smem_set = smem;
  }
  const int units = (a.N / 2) * (a.k_parts > 0 ? a.k_parts : 1);
  const int per_sm = smem > 100 * 1024 ? 1 : 2;
  const int blocks = std::min((units + SM_THREADS / 32 - 1) / (SM_THREADS / 32), n_sms * per_sm);
  return launch_pdl(small_gemm_kernel<KIND, MR, NORM>, dim3(blocks), dim3(SM_THREADS), smem, s, a) == cudaSuccess ? 0 : -1;
}
// the row count is a template argument (rows beyond M would be multiplied as zeros): 1, 4 or 8
template <int KIND, bool NORM>
int launch_small(const SmallArgs& a, int n_sms, cudaStream_t s) {
  if (a.M == 1) return launch_small_mr<KIND, NORM, 1>(a, n_sms, s);
  if (a.M <= 4) return launch_small_mr<KIND, NORM, 4>(a, n_sms, s);
  return launch_small_mr<KIND, NORM, SMALL_GEMM_MAX_ROWS>(a, n_sms, s);
}

}  // namespace

int launch_small_gemm(GemmEpilogueKind kind, const void* epilogue, int M, int N, int K, const float* x_f32,
                      const float* gain, float eps, const __half* a_f16, const __half* w, int gu_blk, int n_sms,
                      cudaStream_t s) {
  if (M <= 0) return 0;
  if (M > SMALL_GEMM_MAX_ROWS || K % 256 != 0 || N % 2 != 0) return -1;
  SmallArgs a{};
  a.M = M; a.N = N; a.K = K; a.x_f32 = x_f32; a.gain = gain; a.eps = eps; a.a_f16 = a_f16; a.w = w; a.gu_blk = gu_blk;
  a.k_parts = 1;
  const bool norm = x_f32 != nullptr;
  switch (kind) {
    case EPI_QKV:
      if (!norm || N % HEAD_DIM != 0) return -1;
      a.qkv = *static_cast<const QkvEpilogue*>(epilogue);
      return launch_small<EPI_QKV, true>(a, n_sms, s);
    case EPI_SWIGLU:
      if (!norm || gu_blk <= 0 || (N / 2) % gu_blk != 0) return -1;
      a.swi = *static_cast<const SwigluEpilogue*>(epilogue);
      return launch_small<EPI_SWIGLU, true>(a, n_sms, s);
    case EPI_RESIDUAL:
      if (norm) return -1;
      a.res = *static_cast<const ResidualEpilogue*>(epilogue);
      // enough warps to keep every SM streaming (sixteen per SM), pieces of whole 256-element strides
      a.k_parts = 1;
      while (a.k_parts < 8 && (N / 2) * a.k_parts < 16 * n_sms && (K / 256) % (2 * a.k_parts) == 0) a.k_parts *= 2;
      return launch_small<EPI_RESIDUAL, false>(a, n_sms, s);
    default:
      return -1;
  }
}

}  // namespace pc
