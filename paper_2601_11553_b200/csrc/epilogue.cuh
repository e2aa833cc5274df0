// What happens to a GEMM accumulator before it reaches memory.  The same device functions serve the
// tcgen05 GEMM (called from its epilogue warps on values read from TMEM) and the plain reference GEMM
// (called from a separate kernel on an fp32 matrix), so both produce identical bytes from identical sums.
#pragma once
#include "kernels.h"

namespace pc {

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_bf162(__nv_bfloat16 a, __nv_bfloat16 b) {
  __nv_bfloat162 h(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Eight columns c0..c0+7 (c0 < 64, multiple of 8) of the low half of one head and the eight columns
// 64 higher, for one row.  `hb` is the head block inside the fused QKV output:
// [0, Hq) query heads, [Hq, Hq+Hkv) key heads, [Hq+Hkv, Hq+2Hkv) value heads.
//   Q: rotate to the row's position, round to fp16, write to q_out.
//   K: round to bf16 (the cache format); keep the unrotated value in the row's page if it has one
//      (paper Section 3.2.1: tensors collected during prefill are saved per chunk); rotate the bf16
//      value to the row's position (Appendix B.1: position counter offset by the cached length) and
//      write it to the assembled context as fp16.
//   V: round to bf16; keep in the page; write to the assembled context.
// The row's position, context slot and page slot are read once per tile by the caller (QkvRow).
struct QkvRow { int pos, slot, pool_tok; };
__device__ __forceinline__ QkvRow load_qkv_row(const QkvEpilogue& e, int row) {
  return QkvRow{__ldg(e.rows.pos + row), __ldg(e.rows.slot + row), __ldg(e.rows.pool_tok + row)};
}
// (cos, sin) of eight consecutive frequencies: read-only path, so the loads may be hoisted above stores
__device__ __forceinline__ void load_cs8(const float2* cs, float2 (&out)[8]) {
  const float4* p = reinterpret_cast<const float4*>(cs);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float4 t = __ldg(p + i);
    out[2 * i] = make_float2(t.x, t.y);
    out[2 * i + 1] = make_float2(t.z, t.w);
  }
}
__device__ __forceinline__ void qkv_store8(const QkvEpilogue& e, int row, const QkvRow& rw, int hb, int c0,
                                           const float (&lo)[8], const float (&hi)[8]) {
  const int pos = rw.pos;
  if (hb < e.n_q_heads) {
    float2 cs[8];
    load_cs8(e.rope + static_cast<size_t>(pos) * ROPE_HALF + c0, cs);
    uint32_t olo[4], ohi[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 a = cs[2 * i], b = cs[2 * i + 1];
      olo[i] = pack_half2(lo[2 * i] * a.x - hi[2 * i] * a.y, lo[2 * i + 1] * b.x - hi[2 * i + 1] * b.y);
      ohi[i] = pack_half2(hi[2 * i] * a.x + lo[2 * i] * a.y, hi[2 * i + 1] * b.x + lo[2 * i + 1] * b.y);
    }
    __half* dst = e.q_out + static_cast<size_t>(row) * (e.n_q_heads * HEAD_DIM) + hb * HEAD_DIM + c0;
    *reinterpret_cast<uint4*>(dst) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
    *reinterpret_cast<uint4*>(dst + ROPE_HALF) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
    return;
  }
  const bool is_k = hb < e.n_q_heads + e.n_kv_heads;
  const int kvh = is_k ? hb - e.n_q_heads : hb - e.n_q_heads - e.n_kv_heads;
  const int kv_dim = e.n_kv_heads * HEAD_DIM;
  const int slot = rw.slot;
  const int ptok = rw.pool_tok;
  __nv_bfloat16 blo[8], bhi[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    blo[i] = __float2bfloat16_rn(lo[i]);
    bhi[i] = __float2bfloat16_rn(hi[i]);
  }
  if (ptok >= 0) {
    __nv_bfloat16* p = (is_k ? e.kpool : e.vpool) + static_cast<size_t>(ptok) * kv_dim + kvh * HEAD_DIM + c0;
    *reinterpret_cast<uint4*>(p) = make_uint4(pack_bf162(blo[0], blo[1]), pack_bf162(blo[2], blo[3]),
                                              pack_bf162(blo[4], blo[5]), pack_bf162(blo[6], blo[7]));
    *reinterpret_cast<uint4*>(p + ROPE_HALF) = make_uint4(pack_bf162(bhi[0], bhi[1]), pack_bf162(bhi[2], bhi[3]),
                                                          pack_bf162(bhi[4], bhi[5]), pack_bf162(bhi[6], bhi[7]));
  }
  uint32_t olo[4], ohi[4];
  if (is_k) {
    float2 cs[8];
    load_cs8(e.rope + static_cast<size_t>(pos) * ROPE_HALF + c0, cs);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 a = cs[2 * i], b = cs[2 * i + 1];
      const float l0 = __bfloat162float(blo[2 * i]), l1 = __bfloat162float(blo[2 * i + 1]);
      const float h0 = __bfloat162float(bhi[2 * i]), h1 = __bfloat162float(bhi[2 * i + 1]);
      olo[i] = pack_half2(l0 * a.x - h0 * a.y, l1 * b.x - h1 * b.y);
      ohi[i] = pack_half2(h0 * a.x + l0 * a.y, h1 * b.x + l1 * b.y);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      olo[i] = pack_half2(__bfloat162float(blo[2 * i]), __bfloat162float(blo[2 * i + 1]));
      ohi[i] = pack_half2(__bfloat162float(bhi[2 * i]), __bfloat162float(bhi[2 * i + 1]));
    }
  }
  __half* dst = (is_k ? e.kctx : e.vctx) + static_cast<size_t>(slot) * kv_dim + kvh * HEAD_DIM + c0;
  *reinterpret_cast<uint4*>(dst) = make_uint4(olo[0], olo[1], olo[2], olo[3]);
  *reinterpret_cast<uint4*>(dst + ROPE_HALF) = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
}

// resid[row][col..col+31] += acc: all loads first, then all stores, so the eight 16-byte accesses overlap
__device__ __forceinline__ void residual_add32(const ResidualEpilogue& e, int row, int col, const uint32_t (&r)[32]) {
  float4* p = reinterpret_cast<float4*>(e.resid + static_cast<size_t>(row) * e.ld + col);
  float4 v[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = p[i];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[i].x += __uint_as_float(r[4 * i]); v[i].y += __uint_as_float(r[4 * i + 1]);
    v[i].z += __uint_as_float(r[4 * i + 2]); v[i].w += __uint_as_float(r[4 * i + 3]);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) p[i] = v[i];
}

// resid[row][col..col+3] += acc
__device__ __forceinline__ void residual_add4(const ResidualEpilogue& e, int row, int col, float a0, float a1,
                                              float a2, float a3) {
  float4* p = reinterpret_cast<float4*>(e.resid + static_cast<size_t>(row) * e.ld + col);
  float4 v = *p;
  v.x += a0; v.y += a1; v.z += a2; v.w += a3;
  *p = v;
}

// act[row][j0..j0+7] = silu(gate) * up, rounded to fp16
__device__ __forceinline__ void swiglu_store8(const SwigluEpilogue& e, int row, int j0, const float (&g)[8],
                                              const float (&u)[8]) {
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = pack_half2(silu_f(g[2 * i]) * u[2 * i], silu_f(g[2 * i + 1]) * u[2 * i + 1]);
  *reinterpret_cast<uint4*>(e.act + static_cast<size_t>(row) * e.ld + j0) = make_uint4(o[0], o[1], o[2], o[3]);
}

}  // namespace pc
