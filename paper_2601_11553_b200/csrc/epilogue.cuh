// What happens to a GEMM accumulator before it reaches memory.  The same device functions serve the
// tcgen05 GEMM (called from its epilogue warps on values read from TMEM) and the plain reference GEMM
// (called from a separate kernel on an fp32 matrix), so both produce identical bytes from identical sums.
#pragma once
#include "kernels.h"
#include "ptx.cuh"

namespace pc {

// x * sigmoid(x); the quotient by the fast reciprocal (1 ulp), not the IEEE division sequence: the result is
// rounded to fp16 right after, and the division was a third of the SwiGLU epilogue's time
__device__ __forceinline__ float silu_f(float x) { return __fdividef(x, 1.0f + __expf(-x)); }

__device__ __forceinline__ uint32_t pack_bf162(__nv_bfloat16 a, __nv_bfloat16 b) {
  __nv_bfloat162 h(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// The row's position, context slot and page slot.
struct QkvRow { int pos, slot, pool_tok; };
__device__ __forceinline__ QkvRow load_qkv_row(const QkvEpilogue& e, int row) {
  return QkvRow{__ldg(e.rows.pos + row), __ldg(e.rows.slot + row), __ldg(e.rows.pool_tok + row)};
}

__device__ __forceinline__ uint2 pack_half4(float a, float b, float c, float d) {
  return make_uint2(pack_half2(a, b), pack_half2(c, d));
}

// Four columns c..c+3 (c < 64, multiple of 4) of the low half of one head and the four columns 64
// higher, for one row.  `hb` is the head block inside the fused QKV output:
// [0, Hq) query heads, [Hq, Hq+Hkv) key heads, [Hq+Hkv, Hq+2Hkv) value heads.
//   Q: rotate to the row's position, round to fp16, write to q_out.
//   K: round to bf16 (the cache format); keep the unrotated value in the row's page if it has one
//      (paper Section 3.2.1: tensors collected during prefill are saved per chunk); rotate the bf16
//      value to the row's position (Appendix B.1: position counter offset by the cached length) and
//      write it to the assembled context as fp16.
//   V: round to bf16; keep in the page; write to the assembled context.
// Callers give adjacent lanes adjacent column groups of the same row, so table reads and stores of
// four lanes cover contiguous 32- to 128-byte pieces.
// (cos, sin) of columns c, c+1 | c+2, c+3 at position pos; the identity for value heads.
struct RopeCs { float4 t0, t1; };
__device__ __forceinline__ RopeCs qkv_load_cs(const QkvEpilogue& e, int pos, int hb, int c) {
  RopeCs r;
  r.t0 = make_float4(1.f, 0.f, 1.f, 0.f);
  r.t1 = r.t0;
  if (hb < e.n_q_heads + e.n_kv_heads) {
    const float4* t = reinterpret_cast<const float4*>(e.rope + static_cast<size_t>(pos) * ROPE_HALF + c);
    r.t0 = __ldg(t);
    r.t1 = __ldg(t + 1);
  }
  return r;
}
__device__ __forceinline__ void qkv_store4_cs(const QkvEpilogue& e, int row, const QkvRow& rw, int hb, int c, float4 lo,
                                              float4 hi, const RopeCs& cs) {
  const bool is_q = hb < e.n_q_heads;
  const bool is_k = !is_q && hb < e.n_q_heads + e.n_kv_heads;
  const float4 t0 = cs.t0, t1 = cs.t1;
  if (e.paged) {
    // Paper-faithful mode (Section 3.2.1: the Q, K and V tensors of the attention module are what is collected;
    // Appendix B.1: position encoding with the counter offset by the cached length): rotate Q and K to the row's
    // position, round everything to bf16 and write it to the row's page slot.  The identity table entries make the
    // same arithmetic a plain copy for V.
    const int q_dim = e.n_q_heads * HEAD_DIM, kv_dim2 = e.n_kv_heads * HEAD_DIM;
    __nv_bfloat16* dst = is_q ? e.qpool + static_cast<size_t>(rw.pool_tok) * q_dim + hb * HEAD_DIM + c
                              : (is_k ? e.kpool + static_cast<size_t>(rw.pool_tok) * kv_dim2 + (hb - e.n_q_heads) * HEAD_DIM + c
                                      : e.vpool + static_cast<size_t>(rw.pool_tok) * kv_dim2 +
                                            (hb - e.n_q_heads - e.n_kv_heads) * HEAD_DIM + c);
    *reinterpret_cast<uint2*>(dst) =
        make_uint2(pack_bf162(__float2bfloat16_rn(lo.x * t0.x - hi.x * t0.y), __float2bfloat16_rn(lo.y * t0.z - hi.y * t0.w)),
                   pack_bf162(__float2bfloat16_rn(lo.z * t1.x - hi.z * t1.y), __float2bfloat16_rn(lo.w * t1.z - hi.w * t1.w)));
    *reinterpret_cast<uint2*>(dst + ROPE_HALF) =
        make_uint2(pack_bf162(__float2bfloat16_rn(hi.x * t0.x + lo.x * t0.y), __float2bfloat16_rn(hi.y * t0.z + lo.y * t0.w)),
                   pack_bf162(__float2bfloat16_rn(hi.z * t1.x + lo.z * t1.y), __float2bfloat16_rn(hi.w * t1.z + lo.w * t1.w)));
    return;
  }
  if (is_q) {
    __half* dst = e.q_out + static_cast<size_t>(row) * (e.n_q_heads * HEAD_DIM) + hb * HEAD_DIM + c;
    *reinterpret_cast<uint2*>(dst) = pack_half4(lo.x * t0.x - hi.x * t0.y, lo.y * t0.z - hi.y * t0.w,
                                                lo.z * t1.x - hi.z * t1.y, lo.w * t1.z - hi.w * t1.w);
    *reinterpret_cast<uint2*>(dst + ROPE_HALF) = pack_half4(hi.x * t0.x + lo.x * t0.y, hi.y * t0.z + lo.y * t0.w,
                                                            hi.z * t1.x + lo.z * t1.y, hi.w * t1.z + lo.w * t1.w);
    return;
  }
  const int kvh = is_k ? hb - e.n_q_heads : hb - e.n_q_heads - e.n_kv_heads;
  const int kv_dim = e.n_kv_heads * HEAD_DIM;
  const __nv_bfloat16 bl0 = __float2bfloat16_rn(lo.x), bl1 = __float2bfloat16_rn(lo.y),
                      bl2 = __float2bfloat16_rn(lo.z), bl3 = __float2bfloat16_rn(lo.w);
  const __nv_bfloat16 bh0 = __float2bfloat16_rn(hi.x), bh1 = __float2bfloat16_rn(hi.y),
                      bh2 = __float2bfloat16_rn(hi.z), bh3 = __float2bfloat16_rn(hi.w);
  if (rw.pool_tok >= 0) {
    __nv_bfloat16* p = (is_k ? e.kpool : e.vpool) + static_cast<size_t>(rw.pool_tok) * kv_dim + kvh * HEAD_DIM + c;
    *reinterpret_cast<uint2*>(p) = make_uint2(pack_bf162(bl0, bl1), pack_bf162(bl2, bl3));
    *reinterpret_cast<uint2*>(p + ROPE_HALF) = make_uint2(pack_bf162(bh0, bh1), pack_bf162(bh2, bh3));
  }
  const float l0 = __bfloat162float(bl0), l1 = __bfloat162float(bl1), l2 = __bfloat162float(bl2),
              l3 = __bfloat162float(bl3);
  const float h0 = __bfloat162float(bh0), h1 = __bfloat162float(bh1), h2 = __bfloat162float(bh2),
              h3 = __bfloat162float(bh3);
  if (e.skip_ctx) return;
  __half* dst = (is_k ? e.kctx : e.vctx) + static_cast<size_t>(rw.slot) * kv_dim + kvh * HEAD_DIM + c;
  if (is_k) {
    *reinterpret_cast<uint2*>(dst) = pack_half4(l0 * t0.x - h0 * t0.y, l1 * t0.z - h1 * t0.w, l2 * t1.x - h2 * t1.y,
                                                l3 * t1.z - h3 * t1.w);
    *reinterpret_cast<uint2*>(dst + ROPE_HALF) = pack_half4(h0 * t0.x + l0 * t0.y, h1 * t0.z + l1 * t0.w,
                                                            h2 * t1.x + l2 * t1.y, h3 * t1.z + l3 * t1.w);
  } else {
    *reinterpret_cast<uint2*>(dst) = pack_half4(l0, l1, l2, l3);
    *reinterpret_cast<uint2*>(dst + ROPE_HALF) = pack_half4(h0, h1, h2, h3);
  }
}

__device__ __forceinline__ void qkv_store4(const QkvEpilogue& e, int row, const QkvRow& rw, int hb, int c, float4 lo,
                                           float4 hi) {
  qkv_store4_cs(e, row, rw, hb, c, lo, hi, qkv_load_cs(e, rw.pos, hb, c));
}

// resid[row][col..col+3] += acc
__device__ __forceinline__ void residual_add4(const ResidualEpilogue& e, int row, int col, float4 a) {
  float4* p = reinterpret_cast<float4*>(e.resid + static_cast<size_t>(row) * e.ld + col);
  float4 v = *p;
  v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
  *p = v;
}

// act[row][j0..j0+3] = silu(gate) * up, rounded to fp16
__device__ __forceinline__ void swiglu_store4(const SwigluEpilogue& e, int row, int j0, float4 g, float4 u) {
  *reinterpret_cast<uint2*>(e.act + static_cast<size_t>(row) * e.ld + j0) =
      pack_half4(silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w);
}

}  // namespace pc
