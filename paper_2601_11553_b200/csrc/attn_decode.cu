// Attention of a decode step: one new row per prompt against that prompt's whole assembled context.
//
// With a single query row per (prompt, KV head) the work is reading K and V once: 512 bytes per context slot and
// KV head for 2 * Hq / Hkv * 128 multiply-adds each, so the kernel is bound by HBM and runs on the CUDA cores (a
// 128-row MMA tile would use one row in 128).  The host cuts every (prompt, KV head) into chunks of context slots,
// one block per chunk; a block keeps the query heads that share the KV head in registers, streams the chunk's K
// and V with 16-byte loads (eight lanes per slot, four slots per warp and step), keeps a running maximum, sum and
// output per slot group (online softmax), folds the groups and warps together, and writes an unnormalised partial
// result; a second kernel merges the chunks of a (prompt, head).  The row at position p sees slots 0..p.
#include <algorithm>

#include "kernels.h"
#include "ptx.cuh"

namespace pc {

namespace {

constexpr int DEC_THREADS = 128;          // 4 warps
constexpr int DEC_WARPS = DEC_THREADS / 32;

__device__ __forceinline__ void half8_to_f32(const uint4& v, float (&f)[8]) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// Where a paged decode step finds K and V: the bf16 pages of one layer, the prompts' page tables (one page id per 16
// slots; an item's ctx0 then is the index of its prompt's first entry) and the (cos, sin) table for rotating K.
struct DecodePages {
  const __nv_bfloat16* kpool;
  const __nv_bfloat16* vpool;
  const int32_t* page_table;
  const float2* rope;
};

// partial_o: [item][group][128] fp32; partial_ml: [item][group][2] (reference maximum in log2 units, sum)
// PAGED = false: K (rotated) and V from the assembled fp16 context; a lane holds 16 consecutive dimensions.
// PAGED = true (after a gather-free prefill): K and V straight from the bf16 pages through the page table, K rotated
// to the slot's position as it is loaded; a lane then holds the 16-byte vector l8 of the head's low half and the one
// of its high half (dimensions 8 l8 .. 8 l8 + 7 and 64 + 8 l8 ..), i.e. eight whole rotation pairs.
template <int GROUP, bool PAGED>
__global__ void __launch_bounds__(DEC_THREADS)
decode_attention_kernel(const DecodeAttnItem* __restrict__ items, const __half* q, const __half* kctx,
                        const __half* vctx, DecodePages pages, float* __restrict__ partial_o,
                        float* __restrict__ partial_ml, int n_q_heads, int n_kv_heads, float scale_log2) {
  __shared__ float sm_o[DEC_WARPS][GROUP][HEAD_DIM];
  __shared__ float sm_ml[DEC_WARPS][GROUP][2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int l8 = lane & 7;                  // which 16 of the 128 dimensions this lane holds
  const int grp = lane >> 3;                // which of the warp's four slots per step
  // first dimension of the lane's two 8-element vectors
  const int d_lo = PAGED ? l8 * 8 : l8 * 16, d_hi = PAGED ? ROPE_HALF + l8 * 8 : l8 * 16 + 8;
  pdl_launch_dependents();
  const DecodeAttnItem it = items[blockIdx.x];     // host-written before the step's first kernel: read ahead of the wait
  pdl_wait();
  const int kv_dim = n_kv_heads * HEAD_DIM;
  const int g = it.kv_head;
  // the query heads of this KV head, 16 dimensions per lane, pre-scaled so that scores come out in log2 units
  float qv[GROUP][16];
#pragma unroll
  for (int h = 0; h < GROUP; ++h) {
    const __half* qp = q + (static_cast<size_t>(it.row) * n_q_heads + g * GROUP + h) * HEAD_DIM;
    float f[8];
    half8_to_f32(ld_dep_v4(qp + d_lo), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) qv[h][e] = f[e] * scale_log2;
    half8_to_f32(ld_dep_v4(qp + d_hi), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) qv[h][8 + e] = f[e] * scale_log2;
  }
  float m[GROUP], l[GROUP], o[GROUP][16];
#pragma unroll
  for (int h = 0; h < GROUP; ++h) {
    m[h] = -INFINITY;
    l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) o[h][e] = 0.f;
  }
  const size_t base = static_cast<size_t>(it.ctx0) * kv_dim + g * HEAD_DIM + l8 * 16;
  // Loads run three steps ahead of the arithmetic (three register buffers), so that every warp keeps 6 KB in flight.
  constexpr int STEP = DEC_WARPS * 4;
  constexpr int NR = 4;
  // Paged form: (cos, sin) of the lane's eight pairs at the slot it works on.  A lane's slots are STEP = 16 apart, so
  // the first comes from the table and every next one is a complex multiplication by the table's row 16 on (a chunk
  // has at most 64 such steps: the error stays near 1e-6 relative).
  float cs[16], cs_step[16];
  if constexpr (PAGED) {
    const float4* c0 = reinterpret_cast<const float4*>(pages.rope + static_cast<size_t>(it.slot_begin + warp * 4 + grp) * ROPE_HALF + l8 * 8);
    const float4* c1 = reinterpret_cast<const float4*>(pages.rope + static_cast<size_t>(STEP) * ROPE_HALF + l8 * 8);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const float4 a = __ldg(c0 + x), b = __ldg(c1 + x);
      cs[4 * x] = a.x; cs[4 * x + 1] = a.y; cs[4 * x + 2] = a.z; cs[4 * x + 3] = a.w;
      cs_step[4 * x] = b.x; cs_step[4 * x + 1] = b.y; cs_step[4 * x + 2] = b.z; cs_step[4 * x + 3] = b.w;
    }
  }
  // Paged form: a lane's slots are 16 apart, i.e. one page-table entry per step; the entries are requested three
  // steps ahead of the loads that need them so that the K/V loads never wait for a table entry.
  int pq0 = 0, pq1 = 0, pq2 = 0;
  int pq_slot = it.slot_begin + warp * 4 + grp;             // slot whose page id pq0 holds
  if constexpr (PAGED) {
    const int32_t* pt = pages.page_table + it.ctx0;
    const int last = (it.slot_end - 1) >> 4;
    pq0 = __ldg(pt + min(pq_slot >> 4, last));
    pq1 = __ldg(pt + min((pq_slot + STEP) >> 4, last));
    pq2 = __ldg(pt + min((pq_slot + 2 * STEP) >> 4, last));
  }
  auto fetch = [&](int s0, uint4 (&r)[NR]) {
    const int slot = s0 + grp;
    int page = 0;
    if constexpr (PAGED) {       // fetches come in slot order, one step apart: pop the queue, request one more entry
      page = pq0;
      pq0 = pq1;
      pq1 = pq2;
      pq_slot += STEP;
      pq2 = __ldg(pages.page_table + it.ctx0 + min((pq_slot + 2 * STEP) >> 4, (it.slot_end - 1) >> 4));
    }
    if (slot < it.slot_end) {
      if constexpr (PAGED) {
        const size_t off = (static_cast<size_t>(page) * PAGE_TOKENS + (slot & 15)) * kv_dim + g * HEAD_DIM;
        r[0] = ld_dep_v4(pages.kpool + off + d_lo);     // the newest slot was written by the kernel before this one
        r[1] = ld_dep_v4(pages.kpool + off + d_hi);
        r[2] = ld_dep_v4(pages.vpool + off + d_lo);
        r[3] = ld_dep_v4(pages.vpool + off + d_hi);
      } else {
        const size_t off = base + static_cast<size_t>(slot) * kv_dim;
        r[0] = ld_dep_v4(kctx + off);          // the newest slot was written by the kernel before this one
        r[1] = ld_dep_v4(kctx + off + 8);
        r[2] = ld_dep_v4(vctx + off);
        r[3] = ld_dep_v4(vctx + off + 8);
      }
    }
  };
  auto consume = [&](int s0, const uint4 (&r)[NR]) {
    const bool live = s0 + grp < it.slot_end;
    float kf[16], vf[16];
    if constexpr (PAGED) {
      float lo[8], hi[8];
      bf16x8_to_f32(r[0], lo);
      bf16x8_to_f32(r[1], hi);
      bf16x8_to_f32(r[2], *reinterpret_cast<float(*)[8]>(&vf[0]));
      bf16x8_to_f32(r[3], *reinterpret_cast<float(*)[8]>(&vf[8]));
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float c = cs[2 * e], sn = cs[2 * e + 1];
        kf[e] = lo[e] * c - hi[e] * sn;
        kf[8 + e] = hi[e] * c + lo[e] * sn;
        cs[2 * e] = c * cs_step[2 * e] - sn * cs_step[2 * e + 1];          // on to the lane's next slot
        cs[2 * e + 1] = sn * cs_step[2 * e] + c * cs_step[2 * e + 1];
      }
    } else {
      half8_to_f32(r[0], *reinterpret_cast<float(*)[8]>(&kf[0]));
      half8_to_f32(r[1], *reinterpret_cast<float(*)[8]>(&kf[8]));
      half8_to_f32(r[2], *reinterpret_cast<float(*)[8]>(&vf[0]));
      half8_to_f32(r[3], *reinterpret_cast<float(*)[8]>(&vf[8]));
    }
#pragma unroll
    for (int h = 0; h < GROUP; ++h) {
      float sc = 0.f;
#pragma unroll
      for (int e = 0; e < 16; ++e) sc = fmaf(qv[h][e], kf[e], sc);
      sc += __shfl_xor_sync(0xffffffffu, sc, 1);
      sc += __shfl_xor_sync(0xffffffffu, sc, 2);
      sc += __shfl_xor_sync(0xffffffffu, sc, 4);          // all eight lanes of the slot hold its score
      if (!live) sc = -INFINITY;
      const float m_new = fmaxf(m[h], sc);
      if (m_new > -INFINITY) {
        const float alpha = exp2f(m[h] - m_new);            // 0 when m was -inf
        const float p = exp2f(sc - m_new);
        l[h] = l[h] * alpha + p;
#pragma unroll
        for (int e = 0; e < 16; ++e) o[h][e] = fmaf(p, live ? vf[e] : 0.f, o[h][e] * alpha);
        m[h] = m_new;
      }
    }
  };
  uint4 ra[NR] = {}, rb[NR] = {}, rc[NR] = {};
  int s0 = it.slot_begin + warp * 4;
  fetch(s0, ra);
  fetch(s0 + STEP, rb);
  fetch(s0 + 2 * STEP, rc);
  while (s0 < it.slot_end) {
    {
      uint4 c[NR];
#pragma unroll
      for (int x = 0; x < NR; ++x) c[x] = ra[x];
      fetch(s0 + 3 * STEP, ra);
      consume(s0, c);
    }
    s0 += STEP;
    if (s0 >= it.slot_end) break;
    {
      uint4 c[NR];
#pragma unroll
      for (int x = 0; x < NR; ++x) c[x] = rb[x];
      fetch(s0 + 3 * STEP, rb);
      consume(s0, c);
    }
    s0 += STEP;
    if (s0 >= it.slot_end) break;
    {
      uint4 c[NR];
#pragma unroll
      for (int x = 0; x < NR; ++x) c[x] = rc[x];
      fetch(s0 + 3 * STEP, rc);
      consume(s0, c);
    }
    s0 += STEP;
  }
  // fold the warp's four slot groups (lanes l8, l8 + 8, l8 + 16, l8 + 24 hold the same dimensions)
#pragma unroll
  for (int h = 0; h < GROUP; ++h) {
#pragma unroll
    for (int x = 8; x <= 16; x <<= 1) {
      const float m_o = __shfl_xor_sync(0xffffffffu, m[h], x);
      const float l_o = __shfl_xor_sync(0xffffffffu, l[h], x);
      const float m_n = fmaxf(m[h], m_o);
      const float a = m[h] > -INFINITY ? exp2f(m[h] - m_n) : 0.f;
      const float b = m_o > -INFINITY ? exp2f(m_o - m_n) : 0.f;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const float o_o = __shfl_xor_sync(0xffffffffu, o[h][e], x);
        o[h][e] = o[h][e] * a + o_o * b;
      }
      l[h] = l[h] * a + l_o * b;
      m[h] = m_n;
    }
    if (grp == 0) {
#pragma unroll
      for (int e = 0; e < 16; ++e) sm_o[warp][h][(e < 8 ? d_lo + e : d_hi + e - 8)] = o[h][e];
      if (l8 == 0) { sm_ml[warp][h][0] = m[h]; sm_ml[warp][h][1] = l[h]; }
    }
  }
  __syncthreads();
  // fold the warps: thread d owns dimension d
  const int d = threadIdx.x;
#pragma unroll
  for (int h = 0; h < GROUP; ++h) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, sm_ml[w][h][0]);
    float acc = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) {
      const float wgt = sm_ml[w][h][0] > -INFINITY ? exp2f(sm_ml[w][h][0] - M) : 0.f;
      acc = fmaf(wgt, sm_o[w][h][d], acc);
      L = fmaf(wgt, sm_ml[w][h][1], L);
    }
    const size_t slot = static_cast<size_t>(it.partial_slot) * GROUP + h;
    partial_o[slot * HEAD_DIM + d] = acc;
    if (d == 0) { partial_ml[slot * 2] = M; partial_ml[slot * 2 + 1] = L; }
  }
}

// out[row][head][:] = sum_c w_c O_c / sum_c w_c l_c over the chunks of (row, KV head), w_c = 2^(m_c - max m).
template <int GROUP>
__global__ void __launch_bounds__(HEAD_DIM)
decode_merge_kernel(const DecodeAttnMerge* __restrict__ merges, const float* partial_o, const float* partial_ml,
                    __half* __restrict__ out, int n_q_heads) {
  pdl_launch_dependents();
  const DecodeAttnMerge mg = merges[blockIdx.x];   // host-written, as above
  pdl_wait();
  const int h = blockIdx.y, d = threadIdx.x;
  // eight parts at a time, all their loads issued before the first is used (a part index past the end repeats the
  // last part and gets weight zero)
  constexpr int U = 8;
  auto slot_of = [&](int c) { return static_cast<size_t>(mg.partial_slot0 + min(c, mg.n_parts - 1)) * GROUP + h; };
  float M = -INFINITY;
  for (int c0 = 0; c0 < mg.n_parts; c0 += U) {
    float mv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) mv[u] = ld_dep_f32(partial_ml + slot_of(c0 + u) * 2);
#pragma unroll
    for (int u = 0; u < U; ++u) M = fmaxf(M, mv[u]);
  }
  float acc = 0.f, L = 0.f;
  for (int c0 = 0; c0 < mg.n_parts; c0 += U) {
    float mv[U], ov[U], lv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t slot = slot_of(c0 + u);
      mv[u] = ld_dep_f32(partial_ml + slot * 2);
      lv[u] = ld_dep_f32(partial_ml + slot * 2 + 1);
      ov[u] = ld_dep_f32(partial_o + slot * HEAD_DIM + d);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const float wgt = (c0 + u < mg.n_parts && mv[u] > -INFINITY) ? exp2f(mv[u] - M) : 0.f;
      acc = fmaf(wgt, ov[u], acc);
      L = fmaf(wgt, lv[u], L);
    }
  }
  out[(static_cast<size_t>(mg.row) * n_q_heads + mg.kv_head * GROUP + h) * HEAD_DIM + d] = to_half_sat(acc / L);
}

}  // namespace

int launch_decode_attention(const DecodeAttnItem* items, int n_items, const DecodeAttnMerge* merges, int n_merges,
                            const __half* q, const __half* kctx_layer, const __half* vctx_layer, float* partial_o,
                            float* partial_ml, __half* out, int n_q_heads, int n_kv_heads, cudaStream_t s,
                            const __nv_bfloat16* kpool_layer, const __nv_bfloat16* vpool_layer,
                            const int32_t* page_table, const float2* rope) {
  if (n_items <= 0) return 0;
  const int group = n_q_heads / n_kv_heads;
  const float scale_log2 = 1.4426950408889634f * 0.08838834764831845f;      // log2(e) / sqrt(128)
  const bool paged = page_table != nullptr;
  if (paged && (!kpool_layer || !vpool_layer || !rope)) return -1;
  const DecodePages pages{kpool_layer, vpool_layer, page_table, rope};
  cudaError_t rc;
  if (group == 2) {
    rc = paged ? launch_pdl(decode_attention_kernel<2, true>, dim3(n_items), dim3(DEC_THREADS), 0, s, items, q, kctx_layer,
                            vctx_layer, pages, partial_o, partial_ml, n_q_heads, n_kv_heads, scale_log2)
               : launch_pdl(decode_attention_kernel<2, false>, dim3(n_items), dim3(DEC_THREADS), 0, s, items, q, kctx_layer,
                            vctx_layer, pages, partial_o, partial_ml, n_q_heads, n_kv_heads, scale_log2);
    if (rc == cudaSuccess)
      rc = launch_pdl(decode_merge_kernel<2>, dim3(n_merges, 2), dim3(HEAD_DIM), 0, s, merges, partial_o, partial_ml, out,
                      n_q_heads);
  } else if (group == 4) {
    rc = paged ? launch_pdl(decode_attention_kernel<4, true>, dim3(n_items), dim3(DEC_THREADS), 0, s, items, q, kctx_layer,
                            vctx_layer, pages, partial_o, partial_ml, n_q_heads, n_kv_heads, scale_log2)
               : launch_pdl(decode_attention_kernel<4, false>, dim3(n_items), dim3(DEC_THREADS), 0, s, items, q, kctx_layer,
                            vctx_layer, pages, partial_o, partial_ml, n_q_heads, n_kv_heads, scale_log2);
    if (rc == cudaSuccess)
      rc = launch_pdl(decode_merge_kernel<4>, dim3(n_merges, 4), dim3(HEAD_DIM), 0, s, merges, partial_o, partial_ml, out,
                      n_q_heads);
  } else {
    return -1;
  }
  return rc == cudaSuccess ? 0 : -1;
}

}  // namespace pc
