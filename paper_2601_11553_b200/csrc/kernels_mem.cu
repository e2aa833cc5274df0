// Memory-bound kernels: gather + re-RoPE of cached pages, RMSNorm, format conversions, page copies.
#include <algorithm>
#include "epilogue.cuh"
#include "kernels.h"
#include "ptx.cuh"

namespace pc {

// ------------------------------------------------------------------------------------------------
// RoPE table: table[p][i] = (cos, sin)(p * theta^(-2i/128)), i in [0, 64).  Angles are formed in
// double so that position 33 023 is as accurate as position 1; the table is then fp32.
// ------------------------------------------------------------------------------------------------
__global__ void build_rope_table_kernel(float2* table, int max_pos, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_pos * ROPE_HALF) return;
  const int p = idx / ROPE_HALF, i = idx % ROPE_HALF;
  const double inv_freq = pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(HEAD_DIM));
  double s, c;
  sincos(static_cast<double>(p) * inv_freq, &s, &c);
  table[idx] = make_float2(static_cast<float>(c), static_cast<float>(s));
}
void launch_build_rope_table(float2* table, int max_pos, double theta, cudaStream_t s) {
  const int n = max_pos * ROPE_HALF;
  build_rope_table_kernel<<<(n + 255) / 256, 256, 0, s>>>(table, max_pos, theta);
}

// ------------------------------------------------------------------------------------------------
// conversions
// ------------------------------------------------------------------------------------------------
__global__ void bf16_to_f16_kernel(const __nv_bfloat16* __restrict__ src, __half* __restrict__ dst, int64_t n) {
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (; i < n; i += stride) dst[i] = to_half_sat(__bfloat162float(src[i]));
}
void launch_bf16_to_f16(const __nv_bfloat16* src, __half* dst, int64_t n, cudaStream_t s) {
  if (n <= 0) return;
  const int blocks = static_cast<int>(std::min<int64_t>((n + 255) / 256, 148 * 16));
  bf16_to_f16_kernel<<<blocks, 256, 0, s>>>(src, dst, n);
}

__global__ void interleave_rows_kernel(const __nv_bfloat16* __restrict__ gate, const __nv_bfloat16* __restrict__ up,
                                       __half* __restrict__ dst, int rows, int cols, int blk) {
  const int64_t n = static_cast<int64_t>(rows) * cols;
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (; i < n; i += stride) {
    const int r = static_cast<int>(i / cols), c = static_cast<int>(i % cols);
    const int b = r / blk, rr = r % blk;
    dst[(static_cast<int64_t>(2 * b) * blk + rr) * cols + c] = to_half_sat(__bfloat162float(gate[i]));
    dst[(static_cast<int64_t>(2 * b + 1) * blk + rr) * cols + c] = to_half_sat(__bfloat162float(up[i]));
  }
}
void launch_interleave_rows_bf16_to_f16(const __nv_bfloat16* gate, const __nv_bfloat16* up, __half* dst, int rows,
                                        int cols, int blk, cudaStream_t s) {
  interleave_rows_kernel<<<148 * 16, 256, 0, s>>>(gate, up, dst, rows, cols, blk);
}

__global__ void bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ src, float* __restrict__ dst, int64_t n) {
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  pdl_launch_dependents();
  pdl_wait();
  for (; i < n; i += stride) dst[i] = __bfloat162float(src[i]);
}
void launch_bf16_to_f32(const __nv_bfloat16* src, float* dst, int64_t n, cudaStream_t s) {
  if (n <= 0) return;
  const int blocks = static_cast<int>(std::min<int64_t>((n + 255) / 256, 148 * 16));
  launch_pdl(bf16_to_f32_kernel, dim3(blocks), dim3(256), 0, s, src, dst, n);
}

// ------------------------------------------------------------------------------------------------
// RMSNorm: out[r][:] = fp16( x[r][:] * rsqrt(mean(x[r]^2) + eps) * gain[:] ), one warp per row.
// ------------------------------------------------------------------------------------------------
// The row stays in registers between the two passes (VPL float4 per lane, d <= 128 * VPL); all loads of a row
// are issued before the first is used.
template <int VPL>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* x, const float* __restrict__ gain,
                                                      __half* __restrict__ out, int M, int d, float eps,
                                                      const int32_t* __restrict__ row_index) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int nv = d >> 2;
  pdl_launch_dependents();
  // the gain is a weight: it is requested before the wait for the kernel that writes x
  float4 g[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int i = lane + 32 * k;
    g[k] = i < nv ? __ldg(reinterpret_cast<const float4*>(gain) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  // which row of x this output row normalises (a host-written list, or the same row)
  const int src_row = (row_index != nullptr && row < M) ? __ldg(row_index + row) : row;
  pdl_wait();
  if (row >= M) return;
  const float4* xr = reinterpret_cast<const float4*>(x + static_cast<size_t>(src_row) * d);
  float4 v[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int i = lane + 32 * k;
    v[k] = i < nv ? ld_dep_f32x4(xr + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < VPL; ++k) ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float inv = rsqrtf(ss / static_cast<float>(d) + eps);
  uint2* o2 = reinterpret_cast<uint2*>(out + static_cast<size_t>(row) * d);
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int i = lane + 32 * k;
    if (i < nv) {
      o2[i] = pack_half4(v[k].x * inv * g[k].x, v[k].y * inv * g[k].y, v[k].z * inv * g[k].z, v[k].w * inv * g[k].w);
    }
  }
}
// Rows of any length: two passes over global memory.
__global__ void __launch_bounds__(256) rmsnorm_long_kernel(const float* x, const float* __restrict__ gain,
                                                           __half* __restrict__ out, int M, int d, float eps,
                                                           const int32_t* __restrict__ row_index) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  pdl_launch_dependents();
  pdl_wait();
  if (row >= M) return;
  const int lane = threadIdx.x & 31;
  const int src_row = row_index != nullptr ? __ldg(row_index + row) : row;
  const float4* xr = reinterpret_cast<const float4*>(x + static_cast<size_t>(src_row) * d);
  const int nv = d >> 2;
  float ss = 0.f;
  for (int i = lane; i < nv; i += 32) {
    const float4 v = ld_dep_f32x4(xr + i);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float inv = rsqrtf(ss / static_cast<float>(d) + eps);
  const float4* g4 = reinterpret_cast<const float4*>(gain);
  uint2* o2 = reinterpret_cast<uint2*>(out + static_cast<size_t>(row) * d);
  for (int i = lane; i < nv; i += 32) {
    const float4 v = ld_dep_f32x4(xr + i);
    const float4 g = g4[i];
    o2[i] = pack_half4(v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
  }
}
void launch_rmsnorm(const float* x, const float* gain, __half* out, int M, int d, float eps, cudaStream_t s,
                    const int32_t* row_index) {
  if (M <= 0) return;
  const dim3 grid((M + 7) / 8), block(256);
  if (d <= 1024) launch_pdl(rmsnorm_kernel<8>, grid, block, 0, s, x, gain, out, M, d, eps, row_index);
  else if (d <= 2048) launch_pdl(rmsnorm_kernel<16>, grid, block, 0, s, x, gain, out, M, d, eps, row_index);
  else launch_pdl(rmsnorm_long_kernel, grid, block, 0, s, x, gain, out, M, d, eps, row_index);
}

// ------------------------------------------------------------------------------------------------
// Gather + re-RoPE (paper Section 3.2.2: matched tensors are loaded and concatenated in order;
// Appendix B.1: position encodings must correspond to the positions in the full sequence).
//
// One block handles one (layer, page item): up to 16 tokens x kv_dim bf16 of K and of V, both
// contiguous in the store and contiguous in the destination.  All traffic is 16-byte vectors.
//   V: converted bf16 -> fp16 (exact for every bf16 value of magnitude >= 2^-14) and copied.
//   K: the vector holding elements [8j, 8j+8) of a head and the one 64 elements higher are rotated
//      together by the token's (cos, sin) row at its position in this prompt, then written as fp16.
// A thread keeps one (token, j) and walks the heads, so it reads its 8 (cos, sin) pairs once.
// Requires kv_dim = n_kv_heads * 128.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void bf16x8_to_float(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint4 float8_to_f16x8(const float (&f)[8]) {
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = pack_half2(f[2 * i], f[2 * i + 1]);   // saturating: bf16 reaches far beyond fp16
  return make_uint4(o[0], o[1], o[2], o[3]);
}

constexpr int GATHER_THREADS = 256;

__global__ void __launch_bounds__(GATHER_THREADS)
gather_rerope_kernel(const GatherItem* __restrict__ items, int n_items, int n_layers,
                     const __nv_bfloat16* __restrict__ kpool, const __nv_bfloat16* __restrict__ vpool,
                     int64_t pool_pages, __half* __restrict__ kctx, __half* __restrict__ vctx, int64_t ctx_cap,
                     int kv_dim, const float2* __restrict__ rope) {
  const int tid = threadIdx.x;
  const int j = tid & 7;              // which 8-element group of the low half
  const int tok = (tid >> 3) & 15;    // token inside the page
  const int hsel = tid >> 7;          // 0..1: heads hsel, hsel + 2, ...
  const int n_heads = kv_dim / HEAD_DIM;
  const int vec_per_row = kv_dim / 8;
  const int64_t n_units = static_cast<int64_t>(n_items) * n_layers;
  pdl_launch_dependents();
  pdl_wait();
  for (int64_t unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
    const int layer = static_cast<int>(unit / n_items);
    const GatherItem it = items[unit % n_items];
    const size_t src_row0 = (static_cast<size_t>(layer) * pool_pages + it.src_page) * PAGE_TOKENS;
    const size_t dst_row0 = static_cast<size_t>(layer) * ctx_cap + it.dst_slot;
    // ---- V: straight conversion copy, fully coalesced
    {
      const uint4* src = reinterpret_cast<const uint4*>(vpool + src_row0 * kv_dim);
      uint4* dst = reinterpret_cast<uint4*>(vctx + dst_row0 * kv_dim);
      const int n_vec = it.n_tok * vec_per_row;
#pragma unroll 4
      for (int v = tid; v < n_vec; v += GATHER_THREADS) {
        float f[8];
        bf16x8_to_float(__ldg(src + v), f);
        dst[v] = float8_to_f16x8(f);
      }
    }
    // ---- K: rotate (lo, hi) vector pairs
    if (tok < it.n_tok) {
      float2 cs[8];
      const float4* csp =
          reinterpret_cast<const float4*>(rope + static_cast<size_t>(it.pos + tok) * ROPE_HALF + j * 8);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float4 t = __ldg(csp + i);
        cs[2 * i] = make_float2(t.x, t.y);
        cs[2 * i + 1] = make_float2(t.z, t.w);
      }
      const __nv_bfloat16* srow = kpool + (src_row0 + tok) * kv_dim;
      __half* drow = kctx + (dst_row0 + tok) * kv_dim;
#pragma unroll 4
      for (int h = hsel; h < n_heads; h += GATHER_THREADS / 128) {
        const int off = h * HEAD_DIM + j * 8;
        float lo[8], hi[8], ol[8], oh[8];
        bf16x8_to_float(__ldg(reinterpret_cast<const uint4*>(srow + off)), lo);
        bf16x8_to_float(__ldg(reinterpret_cast<const uint4*>(srow + off + ROPE_HALF)), hi);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          ol[i] = lo[i] * cs[i].x - hi[i] * cs[i].y;
          oh[i] = hi[i] * cs[i].x + lo[i] * cs[i].y;
        }
        *reinterpret_cast<uint4*>(drow + off) = float8_to_f16x8(ol);
        *reinterpret_cast<uint4*>(drow + off + ROPE_HALF) = float8_to_f16x8(oh);
      }
    }
  }
}
void launch_gather_rerope(const GatherItem* items, int n_items, int n_layers, const __nv_bfloat16* kpool,
                          const __nv_bfloat16* vpool, int64_t pool_pages, __half* kctx, __half* vctx,
                          int64_t ctx_cap, int kv_dim, const float2* rope, cudaStream_t s) {
  if (n_items <= 0) return;
  const int64_t units = static_cast<int64_t>(n_items) * n_layers;
  const int blocks = static_cast<int>(std::min<int64_t>(units, 148 * 8));
  launch_pdl(gather_rerope_kernel, dim3(blocks), dim3(GATHER_THREADS), 0, s, items, n_items, n_layers, kpool, vpool,
             pool_pages, kctx, vctx, ctx_cap, kv_dim, rope);
}

// ------------------------------------------------------------------------------------------------
// chunk [L][n][kv_dim] <-> pages of the store
// ------------------------------------------------------------------------------------------------
__global__ void chunk_pages_copy_kernel(__nv_bfloat16* chunk, __nv_bfloat16* pool, const int32_t* __restrict__ pages,
                                        int n_tokens, int n_layers, int64_t pool_pages, int kv_dim, int to_pool) {
  const int vec_per_row = kv_dim / 8;
  const int64_t n = static_cast<int64_t>(n_layers) * n_tokens * vec_per_row;
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (; i < n; i += stride) {
    const int v = static_cast<int>(i % vec_per_row);
    const int64_t lt = i / vec_per_row;
    const int t = static_cast<int>(lt % n_tokens);
    const int l = static_cast<int>(lt / n_tokens);
    const int page = pages[t / PAGE_TOKENS];
    uint4* pp = reinterpret_cast<uint4*>(pool + ((static_cast<size_t>(l) * pool_pages + page) * PAGE_TOKENS +
                                                 (t % PAGE_TOKENS)) * kv_dim) + v;
    uint4* cp = reinterpret_cast<uint4*>(chunk) + i;
    if (to_pool) *pp = *cp; else *cp = *pp;
  }
}
void launch_chunk_pages_copy(__nv_bfloat16* chunk, __nv_bfloat16* pool, const int32_t* pages, int n_tokens,
                             int n_layers, int64_t pool_pages, int kv_dim, int to_pool, cudaStream_t s) {
  const int64_t n = static_cast<int64_t>(n_layers) * n_tokens * (kv_dim / 8);
  const int blocks = static_cast<int>(std::min<int64_t>((n + 255) / 256, 148 * 16));
  chunk_pages_copy_kernel<<<blocks, 256, 0, s>>>(chunk, pool, pages, n_tokens, n_layers, pool_pages, kv_dim, to_pool);
}

// ------------------------------------------------------------------------------------------------
// Synthetic pool values: SplitMix64 output function on a per-element counter; four 6-bit fields
// summed, centred and scaled by 1/64 (exact in bf16).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t splitmix64_dev(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__global__ void fill_synthetic_kernel(__nv_bfloat16* kpool, __nv_bfloat16* vpool, const int32_t* __restrict__ pages,
                                      int n_tokens, int n_layers, int64_t pool_pages, int kv_dim, uint64_t seed,
                                      uint64_t chunk_id) {
  const int64_t per_layer = static_cast<int64_t>(n_tokens) * kv_dim;
  const int64_t n = 2 * static_cast<int64_t>(n_layers) * per_layer;
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (; i < n; i += stride) {
    const int64_t e = i % per_layer;
    const int64_t wl = i / per_layer;
    const int layer = static_cast<int>(wl % n_layers);
    const int which = static_cast<int>(wl / n_layers);
    const uint64_t base = ((((seed << 20) + chunk_id) * 2ull + which) * 64ull + layer) << 24;
    const uint64_t h = splitmix64_dev(base + static_cast<uint64_t>(e));
    const int sum = static_cast<int>(h & 63) + static_cast<int>((h >> 6) & 63) + static_cast<int>((h >> 12) & 63) +
                    static_cast<int>((h >> 18) & 63);
    const float val = static_cast<float>(sum - 126) * (1.0f / 64.0f);
    const int t = static_cast<int>(e / kv_dim), c = static_cast<int>(e % kv_dim);
    const int page = pages[t / PAGE_TOKENS];
    __nv_bfloat16* pool = which ? vpool : kpool;
    pool[((static_cast<size_t>(layer) * pool_pages + page) * PAGE_TOKENS + (t % PAGE_TOKENS)) * kv_dim + c] =
        __float2bfloat16_rn(val);
  }
}
void launch_fill_synthetic(__nv_bfloat16* kpool, __nv_bfloat16* vpool, const int32_t* pages, int n_tokens,
                           int n_layers, int64_t pool_pages, int kv_dim, uint64_t seed, uint64_t chunk_id,
                           cudaStream_t s) {
  const int64_t n = 2 * static_cast<int64_t>(n_layers) * n_tokens * kv_dim;
  const int blocks = static_cast<int>(std::min<int64_t>((n + 255) / 256, 148 * 16));
  fill_synthetic_kernel<<<blocks, 256, 0, s>>>(kpool, vpool, pages, n_tokens, n_layers, pool_pages, kv_dim, seed,
                                               chunk_id);
}

}  // namespace pc
