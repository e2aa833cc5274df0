// Causal grouped-query flash attention of the new rows against the assembled context, on tcgen05.
//
// Work unit = (tile of up to 128 consecutive new rows of one prompt, one KV head).  The two query heads
// that share the KV head are two 128-row M tiles of the unit: they have the same rows, positions and
// mask and read the same K/V blocks, so every K/V byte fetched into shared memory is used twice.
// The host cuts the units' context ranges into items and deals them to the CTAs so that every CTA gets
// the same number of context blocks; CTA c runs items [cta_first[c], cta_first[c + 1]) in order.
//
// One persistent CTA per SM, 384 threads:
//   warps 0-3  softmax group of query head 2g      (thread = row; TMEM lanes by warp quarter)
//   warps 4-7  softmax group of query head 2g + 1
//   warp 8     TMA producer: Q tiles of both heads, then K and V blocks of 128 context slots into
//              two-stage rings (each block = two 64-column halves in the 128-byte swizzle)
//   warp 9     MMA issuer: S_i = Q_i K^T into TMEM (and, in MODE 2, O_i += P_i V with P_i read from TMEM)
//   warp 10    MODE 0, 1: issuer of O_i += P_i V;  MODE 2: warps 10-11 rotate K (see below)
// TMEM (512 columns), MODE 0 and 1: O_0 [0,128) O_1 [128,256); one S buffer [256,384) that both heads
// take turns with; P_0 [384,448) P_1 [448,512) (16-bit, two per column).  A softmax group copies its S
// block into registers at once and hands the buffer back, so the next S block is computed while the
// exponentials of the current ones run, and a PV product never stands between a group and its next S
// block: S blocks and PV products are issued by two different threads (see the issuers).
// MODE 2 (no warp to spare): S_0 [256,384) S_1 [384,512), P_i over the first 64 columns of S_i, one
// issuer; per head the chain S -> softmax -> PV -> next S is serial and the two heads alternate.
// The running maximum is only raised when the block maximum exceeds it by more than 8 (in log2
// units), which keeps P below 2^8 and makes rescaling of O in TMEM rare.
// A row at position p sees context slots 0..p of its prompt (hit or freshly computed alike).
#include "kernels.h"
#include "ptx.cuh"

namespace pc {

namespace {

constexpr int ATT_THREADS = 384;               // registers are handed out per four warps: warps 10-11 cost nothing more
constexpr int ATT_THREADS_ROT = 384;
constexpr int BLK = 128;                       // rows per tile and context slots per block
constexpr int HALF_TILE_BYTES = BLK * 64 * 2;  // 16 KB: 128 rows x 64 fp16 (one swizzled half)
constexpr int TILE_BYTES = 2 * HALF_TILE_BYTES;
constexpr int KV_STAGES = 2;
constexpr int ATT_SMEM_BYTES = 2 * TILE_BYTES + 2 * KV_STAGES * TILE_BYTES + 1024;
// MODE 2 stages the unrotated K pages of half a block (64 slots) at a time in a ring of two slots: 2 x 16 KB more
constexpr int KRAW_ROWS = 64;
constexpr int KRAW_SLOT_BYTES = 2 * KRAW_ROWS * 128;       // two 64-column halves of 64 rows
constexpr int ATT_SMEM_BYTES_ROT = ATT_SMEM_BYTES + 2 * KRAW_SLOT_BYTES;
constexpr uint32_t TMEM_O0 = 0, TMEM_SX = 256, TMEM_P0 = 384;
constexpr float RESCALE_THRESHOLD = 8.0f;

struct AttnArgs {
  const AttnItem* items;
  const int32_t* cta_first;
  const int32_t* row_pos;
  const int32_t* page_table;      // paged forms: one page id per 16 context slots; an item's ctx0 indexes its prompt's first entry
  const float2* rope;             // MODE 2: (cos, sin)[position][64]
  int32_t rope_rows;              // MODE 2: positions the table covers
  __half* out;
  float* partial_o;
  float* partial_ml;
  int32_t n_q_heads, n_kv_heads;
  float scale_log2;      // log2(e) / sqrt(head_dim)
  int* err_word;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// two fp32 lanes per instruction (packed in a 64-bit register pair)
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

// max(a, b, c) in one instruction (three-input form of max.f32)
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}

// MODE 0: Q from the query buffer, K and V from the assembled context, all fp16.
// MODE 1 (paper-faithful mode): Q, K and V are read straight from the bf16 pages of the store through the prompt's
// page table, one 16-row page per bulk copy (nothing is gathered into a contiguous context first, and K needs no
// rotation because that mode caches it after position encoding); both MMAs run on bf16 operands and P is written to
// TMEM as bf16.
// MODE 2 (gather-free form of the default mode, where the store holds K before rotation): Q from the fp16 query
// buffer; V straight from its pages by bulk copies (the PV MMA then runs on bf16 operands, P as bf16); K is loaded
// from its pages by two extra warps with 16-byte vector loads, rotated to the slot's position in this prompt in fp32
// (paper Appendix B.1: position encodings must be those of the positions in the full sequence) and written as fp16
// straight into the swizzled shared-memory tile the S MMA reads.  Hit tokens are then never copied to a contiguous
// context: the page gather and its write + re-read of every cached K and V byte disappear.
// Everything else is the same kernel.
template <int MODE>
__global__ void __launch_bounds__(ATT_THREADS, 1)
umma_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, AttnArgs args) {
  constexpr bool PAGED = MODE == 1;                  // Q, K, V all by page copies
  constexpr bool PV_BF16 = MODE != 0;                // V comes from the bf16 pages
  constexpr bool SPLIT = MODE != 2;                  // two MMA issuers and the shared S buffer (see the header)
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t q_full, q_empty;
  __shared__ __align__(8) uint64_t k_full[KV_STAGES], k_empty[KV_STAGES], v_full[KV_STAGES], v_empty[KV_STAGES];
  __shared__ __align__(8) uint64_t s_full[2], p_full[2], o_done[2], o_free[2];
  __shared__ __align__(8) uint64_t sx_free;          // the S buffer has been read into registers (4 warps arrive)
  __shared__ __align__(8) uint64_t kraw_full[2], kraw_empty[2];      // MODE 2: the ring of staged, unrotated K pages
  __shared__ uint32_t tmem_base_slot;
  __shared__ int cta_failed;       // set by any role whose bounded wait ran out (or saw another role's error)

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = base;                                   // [2 heads][2 halves][128][64]
  uint8_t* k_smem = base + 2 * TILE_BYTES;                  // [stages][2 halves][128][64]
  uint8_t* v_smem = k_smem + KV_STAGES * TILE_BYTES;
  uint8_t* kraw_smem = v_smem + KV_STAGES * TILE_BYTES;     // MODE 2: [2 slots][2 halves][64][64] bf16

  // The work list and the row positions are written by the host before the first kernel of the call, not by the
  // kernel this one depends on: they are read ahead of the dependency wait, while the prologue runs.
  const int w_begin = args.cta_first[blockIdx.x], w_end = args.cta_first[blockIdx.x + 1];
  AttnItem first_item{};
  if (w_begin < w_end) first_item = args.items[w_begin];
  int first_pos = 0;
  if (warp < 8 && w_begin < w_end) {
    const int r = (warp & 3) * 32 + lane;
    first_pos = args.row_pos[first_item.row0 + (r < first_item.n_rows ? r : first_item.n_rows - 1)];
  }

  if (threadIdx.x == 0) {
    cta_failed = 0;
    mbar_init(&q_full, 1);
    mbar_init(&q_empty, 1);
    for (int s = 0; s < KV_STAGES; ++s) {
      mbar_init(&k_full[s], MODE == 2 ? 2 : 1); mbar_init(&k_empty[s], 1);      // MODE 2: one arrival per rotating warp
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4);
      mbar_init(&o_done[i], 1); mbar_init(&o_free[i], 4);
      mbar_init(&kraw_full[i], 1); mbar_init(&kraw_empty[i], 2);
    }
    mbar_init(&sx_free, 4);
    fence_mbar_init();
  }
  if (warp == 9) {
    tmem_alloc<512>(&tmem_base_slot);
    tmem_relinquish();
  }
  if (warp == 8 && lane == 0) { prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); }
  pdl_launch_dependents();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;
  pdl_wait();                 // Q and the assembled context come from earlier kernels

  const int group = args.n_q_heads / args.n_kv_heads;      // query heads per KV head (even)
  // An item's `unit` = g * pairs + pair covers query heads (g * group + 2 * pair, +1) and KV head g.
  const int pairs = group / 2;

  if (warp == 8 && PAGED) {
    // ---------------------------------------------------------------- TMA producer, paged: the whole warp works.
    // A 128-row tile is eight pages; lane l copies page (l & 7) of 64-column half ((l >> 3) & 1) (and, for Q, of
    // head (l >> 4)): 32 copies for a Q tile pair, 16 each for a K and a V block, all counted by one barrier.
    uint32_t unit_it = 0, kvit = 0;
    bool ok = true;
    const int pg = lane & 7, hf = (lane >> 3) & 1;
    for (int w = w_begin; w < w_end && ok; ++w, ++unit_it) {
      const AttnItem t = w == w_begin ? first_item : args.items[w];
      const int gp = t.unit;
      const int g = gp / pairs, h0 = g * group + 2 * (gp % pairs);
      const int nb = t.blk_end - t.blk_begin;
      const int32_t* pt = args.page_table + t.ctx0;
      // the tile's first row sits at a position that is a multiple of 128 (tiles start at a prompt's first row)
      const int q_page = __ldg(pt + (__ldg(args.row_pos + t.row0) >> 4) + pg);
      ok = mbar_wait(&q_empty, (unit_it & 1u) ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { cta_failed = 1; break; }
      if (lane == 0) mbar_arrive_expect_tx(&q_full, 2 * TILE_BYTES);
      __syncwarp();
      tma_load_2d(q_smem + (lane >> 4) * TILE_BYTES + hf * HALF_TILE_BYTES + pg * (PAGE_TOKENS * 128), &tmQ, &q_full,
                  (h0 + (lane >> 4)) * HEAD_DIM + hf * 64, q_page * PAGE_TOKENS);
      for (int j = 0; j < nb; ++j, ++kvit) {
        const int st = kvit & 1;
        const uint32_t ph = (kvit >> 1) & 1u;
        const int kv_page = __ldg(pt + (t.blk_begin + j) * (BLK / PAGE_TOKENS) + pg);
        ok = mbar_wait(&k_empty[st], ph ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { cta_failed = 1; break; }
        if (lane == 0) mbar_arrive_expect_tx(&k_full[st], TILE_BYTES);
        __syncwarp();
        if (lane < 16)
          tma_load_2d(k_smem + st * TILE_BYTES + hf * HALF_TILE_BYTES + pg * (PAGE_TOKENS * 128), &tmK, &k_full[st],
                      g * HEAD_DIM + hf * 64, kv_page * PAGE_TOKENS);
        ok = mbar_wait(&v_empty[st], ph ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { cta_failed = 1; break; }
        if (lane == 0) mbar_arrive_expect_tx(&v_full[st], TILE_BYTES);
        __syncwarp();
        if (lane < 16)
          tma_load_2d(v_smem + st * TILE_BYTES + hf * HALF_TILE_BYTES + pg * (PAGE_TOKENS * 128), &tmV, &v_full[st],
                      g * HEAD_DIM + hf * 64, kv_page * PAGE_TOKENS);
      }
    }
  } else if (warp == 8 && MODE == 2) {
    // ---------------------------------------------------------------- TMA producer, MODE 2: Q tiles from the query
    // buffer (lanes 0-3, one 128-row box each); per context block the unrotated K pages into the staging ring, half a
    // block (four pages x two 64-column halves = lanes 16-23) at a time, and the V pages into the V ring (lanes 0-15).
    uint32_t unit_it = 0, kvit = 0, rawit = 0;
    bool ok = true;
    const int pg = lane & 7, hf = (lane >> 3) & 1;
    for (int w = w_begin; w < w_end && ok; ++w, ++unit_it) {
      const AttnItem t = w == w_begin ? first_item : args.items[w];
      const int gp = t.unit;
      const int g = gp / pairs, h0 = g * group + 2 * (gp % pairs);
      const int nb = t.blk_end - t.blk_begin;
      const int32_t* pt = args.page_table + t.ctx0;
      ok = mbar_wait(&q_empty, (unit_it & 1u) ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { cta_failed = 1; break; }
      if (lane == 0) mbar_arrive_expect_tx(&q_full, 2 * TILE_BYTES);
      __syncwarp();
      if (lane < 4)
        tma_load_2d(q_smem + (lane >> 1) * TILE_BYTES + (lane & 1) * HALF_TILE_BYTES, &tmQ, &q_full,
                    (h0 + (lane >> 1)) * HEAD_DIM + (lane & 1) * 64, t.row0);
      for (int j = 0; j < nb && ok; ++j, ++kvit) {
        const int st = kvit & 1;
        const uint32_t ph = (kvit >> 1) & 1u;
        const int page = __ldg(pt + (t.blk_begin + j) * (BLK / PAGE_TOKENS) + pg);     // page of rows 16 pg .. 16 pg + 15
        for (int half = 0; half < 2 && ok; ++half, ++rawit) {
          const int slot = rawit & 1;
          ok = mbar_wait(&kraw_empty[slot], ((rawit >> 1) & 1u) ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { cta_failed = 1; break; }
          if (lane == 0) mbar_arrive_expect_tx(&kraw_full[slot], KRAW_SLOT_BYTES);
          __syncwarp();
          // lane 16 + 4 hf + q copies page (4 half + q) of the block: its 64-column half hf, into rows 16 q .. of the slot
          const int src_page = __shfl_sync(0xffffffffu, page, 4 * half + (lane & 3));
          if (lane >= 16 && lane < 24)
            tma_load_2d(kraw_smem + slot * KRAW_SLOT_BYTES + ((lane >> 2) & 1) * (KRAW_ROWS * 128) + (lane & 3) * (PAGE_TOKENS * 128),
                        &tmK, &kraw_full[slot], g * HEAD_DIM + ((lane >> 2) & 1) * 64, src_page * PAGE_TOKENS);
        }
        if (!ok) break;
        ok = mbar_wait(&v_empty[st], ph ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { cta_failed = 1; break; }
        if (lane == 0) mbar_arrive_expect_tx(&v_full[st], TILE_BYTES);
        __syncwarp();
        if (lane < 16)
          tma_load_2d(v_smem + st * TILE_BYTES + hf * HALF_TILE_BYTES + pg * (PAGE_TOKENS * 128), &tmV, &v_full[st],
                      g * HEAD_DIM + hf * 64, page * PAGE_TOKENS);
      }
    }
  } else if (warp >= 10 && MODE == 2) {
    // ---------------------------------------------------------------- K rotated on its way to the S MMA (MODE 2 only:
    // the other forms are launched without these warps).  64 threads: thread (r0 = tid / 8, j = tid % 8) takes rows
    // r0, r0 + 8, ... and, in each, the 16-byte vector j of the head's low half and the one of its high half (elements
    // 8j..8j+7 and 64 + 8j..): together eight rotation pairs.  It reads them from the staged pages, rotates in fp32 and
    // writes fp16 to the place the 128-byte swizzle gives vector j of that row (j ^ (row & 7)) in both 64-column halves
    // of the K tile.  The (cos, sin) of a block's first eight rows come from the table (requested one block ahead);
    // every further row group is eight positions on, i.e. one more complex multiplication by the table's row 8 --
    // sixteen steps at most before the table is read again.
    if constexpr (MODE == 2) {
      const int tid = (warp - 10) * 32 + lane;
      const int j = tid & 7, r0 = tid >> 3;
      uint32_t kvit = 0, rawit = 0;
      bool ok = true;
      float step[16];                                      // (cos, sin) of 8 positions for this thread's eight pairs
      {
        const float4* sp = reinterpret_cast<const float4*>(args.rope + static_cast<size_t>(min(8, args.rope_rows - 1)) * ROPE_HALF + j * 8);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 v = __ldg(sp + q);
          step[4 * q] = v.x; step[4 * q + 1] = v.y; step[4 * q + 2] = v.z; step[4 * q + 3] = v.w;
        }
      }
      auto load_cs = [&](int pos, float (&cs)[16]) {
        const float4* csp = reinterpret_cast<const float4*>(args.rope + static_cast<size_t>(min(pos, args.rope_rows - 1)) * ROPE_HALF + j * 8);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 v = __ldg(csp + q);
          cs[4 * q] = v.x; cs[4 * q + 1] = v.y; cs[4 * q + 2] = v.z; cs[4 * q + 3] = v.w;
        }
      };
      float cs_next[16];
      if (w_begin < w_end) load_cs(first_item.blk_begin * BLK + r0, cs_next);
      for (int w = w_begin; w < w_end && ok; ++w) {
        const AttnItem t = w == w_begin ? first_item : args.items[w];
        const int nb = t.blk_end - t.blk_begin;
        for (int jb = 0; jb < nb && ok; ++jb, ++kvit) {
          const int st = kvit & 1;
          const uint32_t ph = (kvit >> 1) & 1u;
          float cs[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) cs[q] = cs_next[q];
          // the table row the next block starts from (the next item's first block when this one ends)
          if (jb + 1 < nb) load_cs((t.blk_begin + jb + 1) * BLK + r0, cs_next);
          else if (w + 1 < w_end) load_cs(args.items[w + 1].blk_begin * BLK + r0, cs_next);
          ok = mbar_wait(&k_empty[st], ph ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { cta_failed = 1; break; }
          uint8_t* tile = k_smem + st * TILE_BYTES;
          for (int half = 0; half < 2 && ok; ++half, ++rawit) {
            const int slot = rawit & 1;
            ok = mbar_wait(&kraw_full[slot], (rawit >> 1) & 1u, args.err_word, DEV_ERR_ATTN_PRODUCER);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { cta_failed = 1; break; }
            const uint8_t* raw = kraw_smem + slot * KRAW_SLOT_BYTES;
#pragma unroll 2
            for (int rr = 0; rr < KRAW_ROWS / 8; ++rr) {
              const int rl = r0 + 8 * rr;                      // row inside the staged half block
              const int row = half * KRAW_ROWS + rl;           // row inside the K tile
              const int off = rl * 128 + ((j ^ (rl & 7)) << 4);
              const uint4 vlo = *reinterpret_cast<const uint4*>(raw + off);
              const uint4 vhi = *reinterpret_cast<const uint4*>(raw + KRAW_ROWS * 128 + off);
              const uint32_t wl[4] = {vlo.x, vlo.y, vlo.z, vlo.w}, wh[4] = {vhi.x, vhi.y, vhi.z, vhi.w};
              uint32_t ol[4], oh[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {          // two bf16 elements per 32-bit word
                const float l0 = __uint_as_float(wl[q] << 16), l1 = __uint_as_float(wl[q] & 0xffff0000u);
                const float h0 = __uint_as_float(wh[q] << 16), h1 = __uint_as_float(wh[q] & 0xffff0000u);
                const float ca = cs[4 * q], sa = cs[4 * q + 1], cb = cs[4 * q + 2], sb = cs[4 * q + 3];
                ol[q] = pack_half2(l0 * ca - h0 * sa, l1 * cb - h1 * sb);
                oh[q] = pack_half2(h0 * ca + l0 * sa, h1 * cb + l1 * sb);
              }
              uint8_t* dst = tile + row * 128 + ((j ^ (row & 7)) << 4);
              *reinterpret_cast<uint4*>(dst) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
              *reinterpret_cast<uint4*>(dst + HALF_TILE_BYTES) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
#pragma unroll
              for (int q = 0; q < 8; ++q) {          // eight positions on: (c, s) <- (c, s) * (c8, s8)
                const float c = cs[2 * q], sn = cs[2 * q + 1];
                cs[2 * q] = c * step[2 * q] - sn * step[2 * q + 1];
                cs[2 * q + 1] = sn * step[2 * q] + c * step[2 * q + 1];
              }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&kraw_empty[slot]);     // both warps have read the slot: it may be refilled
          }
          if (!ok) break;
          fence_proxy_async_smem();            // the MMA reads the tile through the async proxy
          __syncwarp();
          if (lane == 0) mbar_arrive(&k_full[st]);
        }
      }
    }
  } else if (warp == 8) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t unit_it = 0, kvit = 0;
      bool ok = true;
      for (int w = w_begin; w < w_end && ok; ++w, ++unit_it) {
        const AttnItem t = w == w_begin ? first_item : args.items[w];
        const int gp = t.unit;
        const int g = gp / pairs, h0 = g * group + 2 * (gp % pairs);
        const int nb = t.blk_end - t.blk_begin;
        if (!mbar_wait(&q_empty, (unit_it & 1u) ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER)) { ok = false; cta_failed = 1; break; }
        mbar_arrive_expect_tx(&q_full, 2 * TILE_BYTES);
        for (int i = 0; i < 2; ++i)
          for (int hf = 0; hf < 2; ++hf)
            tma_load_2d(q_smem + i * TILE_BYTES + hf * HALF_TILE_BYTES, &tmQ, &q_full, (h0 + i) * HEAD_DIM + hf * 64,
                        t.row0);
        for (int j = 0; j < nb; ++j, ++kvit) {
          const int st = kvit & 1;
          const uint32_t ph = (kvit >> 1) & 1u;
          if (!mbar_wait(&k_empty[st], ph ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER)) { ok = false; cta_failed = 1; break; }
          mbar_arrive_expect_tx(&k_full[st], TILE_BYTES);
          for (int hf = 0; hf < 2; ++hf)
            tma_load_2d(k_smem + st * TILE_BYTES + hf * HALF_TILE_BYTES, &tmK, &k_full[st], g * HEAD_DIM + hf * 64,
                        t.ctx0 + (t.blk_begin + j) * BLK);
          if (!mbar_wait(&v_empty[st], ph ^ 1u, args.err_word, DEV_ERR_ATTN_PRODUCER)) { ok = false; cta_failed = 1; break; }
          mbar_arrive_expect_tx(&v_full[st], TILE_BYTES);
          for (int hf = 0; hf < 2; ++hf)
            tma_load_2d(v_smem + st * TILE_BYTES + hf * HALF_TILE_BYTES, &tmV, &v_full[st], g * HEAD_DIM + hf * 64,
                        t.ctx0 + (t.blk_begin + j) * BLK);
        }
      }
      (void)ok;
    }
  } else if (warp == 9 || (warp == 10 && MODE != 2)) {
    // ---------------------------------------------------------------- MMA issuers
    // Issuing a tcgen05.mma holds the thread until the tensor pipe takes it, so a single thread that also polls the
    // barriers between groups leaves the pipe idle for that long after every group.  Where a warp is free (MODE 0
    // and 1) the S blocks are issued by warp 9 and the PV products by warp 10, each in its own order
    // (S_0(j), S_1(j), S_0(j+1), ... and PV_0(j), PV_1(j), ...): every dependency between them goes through a
    // barrier (S buffer free, P written, PV complete), none through the order in the pipe.  In MODE 2 warps 10-11
    // rotate K and warp 9 issues both, in the order  PV_0(j), S_0(j+1), PV_1(j), S_1(j+1).
    if (lane == 0) {
      // operand type of each MMA: 0 fp16, 1 bf16 (both operands of one MMA always have the same type)
      constexpr uint32_t idesc_qk = make_idesc_f16(BLK, BLK, PAGED ? 1 : 0, 0, 0);          // A, B K-major
      constexpr uint32_t idesc_pv = make_idesc_f16(BLK, HEAD_DIM, PV_BF16 ? 1 : 0, 0, 1);   // B (V) MN-major
      uint32_t unit_it = 0, kvit = 0, s_it = 0;      // s_it: S blocks issued so far, all into the one S buffer
      bool ok = true;
      auto fail = [&]() { ok = false; cta_failed = 1; };
      // S_i(kvidx) = Q_i K(kvidx)^T, once the previous S block (of the other head) has been read out of the buffer
      auto issue_s = [&](int i, uint32_t kvidx) {
        if (SPLIT) {
          if (s_it != 0 && !mbar_wait(&sx_free, (s_it - 1u) & 1u, args.err_word, DEV_ERR_ATTN_MMA)) { fail(); return; }
          tc_fence_after_sync();
        }
        const int st = kvidx & 1;
        const uint32_t qa = smem_u32(q_smem + i * TILE_BYTES), ka = smem_u32(k_smem + st * TILE_BYTES);
#pragma unroll
        for (int kk = 0; kk < HEAD_DIM / 16; ++kk) {
          const uint32_t off = (kk >> 2) * HALF_TILE_BYTES + (kk & 3) * 32;
          umma_ss(tmem_base + TMEM_SX + (SPLIT ? 0 : i * BLK), make_smem_desc_sw128(qa + off, 16, 1024),
                  make_smem_desc_sw128(ka + off, 16, 1024), idesc_qk, kk != 0 ? 1u : 0u);
        }
        umma_commit(&s_full[i]);
        ++s_it;
      };
      // O_i += P_i(kvidx) V(kvidx)
      auto issue_pv = [&](int i, uint32_t kvidx, bool first) {
        const int st = kvidx & 1;
        if (!mbar_wait(&p_full[i], kvidx & 1u, args.err_word, DEV_ERR_ATTN_MMA)) { fail(); return; }
        if (first && !mbar_wait(&o_free[i], (unit_it & 1u) ^ 1u, args.err_word, DEV_ERR_ATTN_MMA)) { fail(); return; }
        if (i == 0 && !mbar_wait(&v_full[st], (kvidx >> 1) & 1u, args.err_word, DEV_ERR_ATTN_MMA)) { fail(); return; }
        tc_fence_after_sync();
        const uint32_t va = smem_u32(v_smem + st * TILE_BYTES);
#pragma unroll
        for (int kk = 0; kk < BLK / 16; ++kk) {
          // 16 context slots = 16 rows of 128 bytes in each 64-column half; halves are 16 KB apart
          umma_ts(tmem_base + TMEM_O0 + i * HEAD_DIM, tmem_base + (SPLIT ? TMEM_P0 + i * (BLK / 2) : TMEM_SX + i * BLK) + kk * 8,
                  make_smem_desc_sw128(va + kk * 2048, HALF_TILE_BYTES, 1024), idesc_pv, (!first || kk != 0) ? 1u : 0u);
        }
        umma_commit(&o_done[i]);
        if (i == 1) umma_commit(&v_empty[st]);
      };
      auto wait_k = [&](uint32_t kvidx) {
        if (!mbar_wait(&k_full[kvidx & 1], (kvidx >> 1) & 1u, args.err_word, DEV_ERR_ATTN_MMA)) fail();
      };
      for (int w = w_begin; w < w_end && ok; ++w, ++unit_it) {
        const AttnItem t = w == w_begin ? first_item : args.items[w];
        const int nb = t.blk_end - t.blk_begin;
        const uint32_t kv0 = kvit;
        if (SPLIT && warp == 10) {
          for (int j = 0; j < nb && ok; ++j) {
            issue_pv(0, kv0 + j, j == 0);
            if (ok) issue_pv(1, kv0 + j, j == 0);
          }
          kvit += nb;
          continue;
        }
        if (!mbar_wait(&q_full, unit_it & 1u, args.err_word, DEV_ERR_ATTN_MMA)) { fail(); break; }
        if (SPLIT) {
          for (int j = 0; j < nb && ok; ++j) {
            wait_k(kv0 + j);
            if (ok) issue_s(0, kv0 + j);
            if (ok) issue_s(1, kv0 + j);
            if (!ok) break;
            umma_commit(&k_empty[(kv0 + j) & 1]);
            if (j + 1 == nb) umma_commit(&q_empty);
          }
          kvit += nb;
          continue;
        }
        // one issuer, one S buffer per head: per head the chain S -> softmax -> PV -> next S is serial (P lies over
        // the first half of S), the two heads alternate
        wait_k(kv0);
        if (!ok) break;
        issue_s(0, kv0);
        issue_s(1, kv0);
        umma_commit(&k_empty[kv0 & 1]);
        if (nb == 1) umma_commit(&q_empty);
        for (int j = 0; j < nb && ok; ++j) {
          const uint32_t kvidx = kv0 + j;
          for (int i = 0; i < 2 && ok; ++i) {
            issue_pv(i, kvidx, j == 0);
            if (!ok) break;
            if (j + 1 < nb) {
              if (i == 0) wait_k(kvidx + 1);
              if (!ok) break;
              issue_s(i, kvidx + 1);
              if (i == 1) {
                umma_commit(&k_empty[(kvidx + 1) & 1]);
                if (j + 2 == nb) umma_commit(&q_empty);
              }
            }
          }
        }
        kvit += nb;
      }
    }
  } else if (warp < 8) {
    // ---------------------------------------------------------------- softmax groups (warps 0..7)
    const int i = warp >> 2;                      // which query head of the pair
    const int quarter = warp & 3;
    const int r_in_tile = quarter * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t t_s = tmem_base + lane_base + TMEM_SX + (SPLIT ? 0 : i * BLK);
    const uint32_t t_p = SPLIT ? tmem_base + lane_base + TMEM_P0 + i * (BLK / 2) : t_s;
    const uint32_t t_o = tmem_base + lane_base + TMEM_O0 + i * HEAD_DIM;
    uint32_t unit_it = 0, kvit = 0;
    bool ok = true;
    for (int w = w_begin; w < w_end && ok; ++w, ++unit_it) {
      const AttnItem t = w == w_begin ? first_item : args.items[w];
      const int gp = t.unit;
      const int head = (gp / pairs) * group + 2 * (gp % pairs) + i;
      const int nb = t.blk_end - t.blk_begin;
      const uint32_t kv0 = kvit;
      const bool valid = r_in_tile < t.n_rows;
      const int row = t.row0 + (valid ? r_in_tile : t.n_rows - 1);
      const int pos = w == w_begin ? first_pos : args.row_pos[row];
      float m = -INFINITY, l = 0.f;
      for (int j = 0; j < nb; ++j) {
        const uint32_t kvidx = kv0 + j;
        ok = mbar_wait(&s_full[i], kvidx & 1u, args.err_word, DEV_ERR_ATTN_SOFTMAX);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { cta_failed = 1; break; }
        tc_fence_after_sync();
        uint32_t s[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld_32x32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
        tmem_wait_ld();
        if (SPLIT) {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sx_free);              // the block is in registers: the buffer may take the next
        }
        const int limit = pos - (t.blk_begin + j) * BLK;     // columns 0..limit are visible
        // maximum of the raw scores (the scale is positive, so it commutes with the maximum)
        // four independent chains: the reduction is bound by instruction latency, not by issue
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
        if (limit < BLK - 1) {
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c > limit) s[c] = 0xff800000u;                // -inf
        }
#pragma unroll
        for (int c = 0; c < 128; c += 8) {
          mx0 = fmax3(mx0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
          mx1 = fmax3(mx1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
          mx2 = fmax3(mx2, __uint_as_float(s[c + 4]), __uint_as_float(s[c + 5]));
          mx3 = fmax3(mx3, __uint_as_float(s[c + 6]), __uint_as_float(s[c + 7]));
        }
        const float m_raw = fmax3(fmaxf(mx0, mx1), mx2, mx3);
        const float m_blk = m_raw * args.scale_log2;
        if (j == 0) {
          // an item that starts past the row's position sees nothing: keep a finite reference
          m = m_blk == -INFINITY ? 0.f : m_blk;
        } else {
          const bool need = m_blk > m + RESCALE_THRESHOLD;
          if (__any_sync(0xffffffffu, need)) {
            // O_i must be complete up to the previous block before it is rescaled in place
            ok = mbar_wait(&o_done[i], (kvidx - 1u) & 1u, args.err_word, DEV_ERR_ATTN_CORR);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { cta_failed = 1; break; }
            tc_fence_after_sync();
            float alpha = 1.0f;
            if (need) { alpha = fast_exp2(m - m_blk); m = m_blk; l *= alpha; }
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              uint32_t o[32];
              tmem_ld_32x32(t_o + c * 32, o);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
              tmem_st_32x32(t_o + c * 32, o);
            }
            tmem_wait_st();
          }
        }
        uint32_t p[64];
        const float neg_m = -m;
        const uint64_t scale2 = pack_f32x2(args.scale_log2, args.scale_log2), negm2 = pack_f32x2(neg_m, neg_m);
        uint64_t sum2a = pack_f32x2(0.f, 0.f), sum2b = sum2a;
#pragma unroll
        for (int c = 0; c < 64; ++c) {
          float x0, x1;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[2 * c]), __uint_as_float(s[2 * c + 1])), scale2, negm2), x0, x1);
          const float p0 = fast_exp2(x0);
          const float p1 = fast_exp2(x1);
          if (c & 1) sum2b = add_f32x2(sum2b, pack_f32x2(p0, p1));
          else sum2a = add_f32x2(sum2a, pack_f32x2(p0, p1));
          if constexpr (PV_BF16) {          // P in the operand type of V
            __nv_bfloat162 bb = __floats2bfloat162_rn(p0, p1);
            p[c] = *reinterpret_cast<uint32_t*>(&bb);
          } else {
            __half2 hh = __floats2half2_rn(p0, p1);
            p[c] = *reinterpret_cast<uint32_t*>(&hh);
          }
        }
        float sum0, sum1;
        unpack_f32x2(add_f32x2(sum2a, sum2b), sum0, sum1);
        const float sum = sum0 + sum1;
        l += sum;
        // P_i of the previous block must have been consumed (PV complete) before it is overwritten
        ok = mbar_wait(&o_done[i], (kvidx - 1u) & 1u, args.err_word, DEV_ERR_ATTN_CORR);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { cta_failed = 1; break; }
        tc_fence_after_sync();
        tmem_st_32x32(t_p, *reinterpret_cast<uint32_t(*)[32]>(&p[0]));
        tmem_st_32x32(t_p + 32, *reinterpret_cast<uint32_t(*)[32]>(&p[32]));
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[i]);
      }
      if (!ok) break;
      // ---- final: O_i / l -> fp16 -> out, or the unnormalised part -> scratch
      ok = mbar_wait(&o_done[i], (kv0 + nb - 1u) & 1u, args.err_word, DEV_ERR_ATTN_CORR);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { cta_failed = 1; break; }
      tc_fence_after_sync();
      if (t.partial_slot < 0) {
        const float inv_l = 1.0f / l;
        __half* dst = args.out + (static_cast<size_t>(row) * args.n_q_heads + head) * HEAD_DIM;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld_32x32(t_o + c * 32, o);
          tmem_wait_ld();
          if (valid) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              uint32_t pk[4];
#pragma unroll
              for (int q = 0; q < 4; ++q)     // saturating: P is rounded but the row sum is not, so a quotient of
                                              // values at the fp16 limit can land just beyond it
                pk[q] = pack_half2(__uint_as_float(o[8 * e + 2 * q]) * inv_l, __uint_as_float(o[8 * e + 2 * q + 1]) * inv_l);
              *reinterpret_cast<uint4*>(dst + c * 32 + e * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
          }
        }
      } else {
        const size_t slot = static_cast<size_t>(t.partial_slot) * 2 + i;
        float* po = args.partial_o + (slot * BLK + r_in_tile) * HEAD_DIM;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld_32x32(t_o + c * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 8; ++e)
            *reinterpret_cast<uint4*>(po + c * 32 + e * 4) = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
        }
        // a row that saw nothing in this part contributes nothing: l = 0 and reference -inf
        *reinterpret_cast<float2*>(args.partial_ml + (slot * BLK + r_in_tile) * 2) =
            make_float2(l > 0.f ? m : -INFINITY, l);
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_free[i]);
      kvit += nb;
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (cta_failed) {
    // Error path only (the flag was written before the barrier, so the branch is uniform): let bulk copies this CTA
    // issued land before its shared memory is released, whichever role it was that gave up.
    if (threadIdx.x == 0) {
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < DRAIN_LIMIT_NS) { }
    }
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after_sync();
    tmem_dealloc<512>(tmem_base);
  }
}

}  // namespace

int make_attn_maps(AttnMaps* out, const __half* q, int64_t m_cap, int q_dim, const __half* kctx_layer,
                   const __half* vctx_layer, int64_t ctx_cap, int kv_dim) {
  const uint32_t box[2] = {64u, static_cast<uint32_t>(BLK)};
  {
    const uint64_t dims[2] = {static_cast<uint64_t>(q_dim), static_cast<uint64_t>(m_cap)};
    const uint64_t str[1] = {static_cast<uint64_t>(q_dim) * 2};
    if (encode_f16_map(&out->q, q, 2, dims, str, box) != 0) return -1;
  }
  const uint64_t dims[2] = {static_cast<uint64_t>(kv_dim), static_cast<uint64_t>(ctx_cap)};
  const uint64_t str[1] = {static_cast<uint64_t>(kv_dim) * 2};
  if (encode_f16_map(&out->k, kctx_layer, 2, dims, str, box) != 0) return -1;
  if (encode_f16_map(&out->v, vctx_layer, 2, dims, str, box) != 0) return -1;
  return 0;
}

// Merge of the parts of a split unit: out[row][head] = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s with
// M = max_s m_s.  A warp takes MERGE_ROWS rows of one (unit, head) at a time: for each row, lane s holds part s's
// (reference, sum) pair and its weight, every lane owns four output columns, and the loads of up to four parts
// of all the warp's rows are in flight together (the kernel is a chain of short dependent loads otherwise).
namespace {
constexpr int MERGE_WARPS = 8;
constexpr int MERGE_ROWS = 2;
__global__ void __launch_bounds__(MERGE_WARPS * 32)
attention_merge_kernel(const AttnMerge* __restrict__ merges, const float* partial_o, const float* partial_ml,
                       __half* __restrict__ out, int n_q_heads, int n_kv_heads) {
  pdl_launch_dependents();
  const AttnMerge mg = merges[blockIdx.x];      // host-written before the call's first kernel: read ahead of the wait
  pdl_wait();
  const int group = n_q_heads / n_kv_heads, pairs = group / 2;
  const int i = blockIdx.y;
  const int head = (mg.unit / pairs) * group + 2 * (mg.unit % pairs) + i;
  const int lane = threadIdx.x & 31;
  const int r0 = (blockIdx.z * MERGE_WARPS + (threadIdx.x >> 5)) * MERGE_ROWS;
  if (r0 >= mg.n_rows) return;
  const size_t slot0 = static_cast<size_t>(mg.partial_slot0) * 2 + i;     // part s is two slots further each
  float w[MERGE_ROWS], inv[MERGE_ROWS];
  float4 acc[MERGE_ROWS];
#pragma unroll
  for (int k = 0; k < MERGE_ROWS; ++k) {
    const int r = min(r0 + k, mg.n_rows - 1);
    float2 ml = make_float2(-INFINITY, 0.f);
    if (lane < mg.n_parts) ml = ld_dep_f32x2(partial_ml + ((slot0 + 2 * lane) * BLK + r) * 2);
    float M = ml.y > 0.f ? ml.x : -INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    w[k] = ml.y > 0.f ? exp2f(ml.x - M) : 0.f;
    float l = w[k] * ml.y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    inv[k] = 1.0f / l;
    acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int s0 = 0; s0 < mg.n_parts; s0 += 4) {          // n_parts <= 32: the weights live in lanes 0..n_parts-1
    float4 o[MERGE_ROWS][4];
#pragma unroll
    for (int k = 0; k < MERGE_ROWS; ++k) {
      const int r = min(r0 + k, mg.n_rows - 1);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int sp = min(s0 + q, mg.n_parts - 1);       // a repeated part gets weight zero below
        o[k][q] = ld_dep_f32x4(partial_o + ((slot0 + 2 * sp) * BLK + r) * HEAD_DIM + lane * 4);
      }
    }
#pragma unroll
    for (int k = 0; k < MERGE_ROWS; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float ws = __shfl_sync(0xffffffffu, w[k], (s0 + q) & 31);
        if (s0 + q >= mg.n_parts) ws = 0.f;
        acc[k].x = fmaf(ws, o[k][q].x, acc[k].x); acc[k].y = fmaf(ws, o[k][q].y, acc[k].y);
        acc[k].z = fmaf(ws, o[k][q].z, acc[k].z); acc[k].w = fmaf(ws, o[k][q].w, acc[k].w);
      }
  }
#pragma unroll
  for (int k = 0; k < MERGE_ROWS; ++k) {
    if (r0 + k >= mg.n_rows) break;
    *reinterpret_cast<uint2*>(out + (static_cast<size_t>(mg.row0 + r0 + k) * n_q_heads + head) * HEAD_DIM + lane * 4) =
        make_uint2(pack_half2(acc[k].x * inv[k], acc[k].y * inv[k]), pack_half2(acc[k].z * inv[k], acc[k].w * inv[k]));
  }
}
}  // namespace

void launch_attention_merge(const AttnMerge* merges, int n_merges, const float* partial_o, const float* partial_ml,
                            __half* out, int n_q_heads, int n_kv_heads, cudaStream_t s) {
  if (n_merges <= 0) return;
  dim3 grid(n_merges, 2, BLK / (MERGE_WARPS * MERGE_ROWS));
  launch_pdl(attention_merge_kernel, grid, dim3(MERGE_WARPS * 32), 0, s, merges, partial_o, partial_ml, out, n_q_heads,
             n_kv_heads);
}

int make_paged_attn_maps(AttnMaps* out, const __nv_bfloat16* qpool_layer, const __nv_bfloat16* kpool_layer,
                         const __nv_bfloat16* vpool_layer, int64_t pool_pages, int q_dim, int kv_dim) {
  // one page (16 rows) of a 64-column half per copy; the element type only matters for out-of-range fill, which
  // never happens here (page ids and columns are always inside the pool)
  const uint32_t box[2] = {64u, static_cast<uint32_t>(PAGE_TOKENS)};
  const uint64_t rows = static_cast<uint64_t>(pool_pages) * PAGE_TOKENS;
  const uint64_t qd[2] = {static_cast<uint64_t>(q_dim), rows}, qs[1] = {static_cast<uint64_t>(q_dim) * 2};
  const uint64_t kd[2] = {static_cast<uint64_t>(kv_dim), rows}, ks[1] = {static_cast<uint64_t>(kv_dim) * 2};
  if (encode_f16_map(&out->q, qpool_layer, 2, qd, qs, box) != 0) return -1;
  if (encode_f16_map(&out->k, kpool_layer, 2, kd, ks, box) != 0) return -1;
  if (encode_f16_map(&out->v, vpool_layer, 2, kd, ks, box) != 0) return -1;
  return 0;
}

int launch_umma_attention(const AttnMaps& maps, const AttnItem* items, const int32_t* cta_first, int n_ctas,
                          const int32_t* row_pos, __half* out, float* partial_o, float* partial_ml, int n_q_heads,
                          int n_kv_heads, int* err_word, cudaStream_t s, const int32_t* page_table, int mode,
                          const float2* rope, int rope_rows) {
  if (n_ctas <= 0) return 0;
  const int group = n_q_heads / n_kv_heads;
  if (group < 2 || group % 2 != 0 || mode < 0 || mode > 2) return -1;
  if (mode != 0 && page_table == nullptr) return -1;
  if (mode == 2 && (rope == nullptr || rope_rows <= 8)) return -1;
  static bool smem_set[3][MAX_DEVICES] = {};   // once per device: the call costs host time on every launch otherwise
  const int dev = current_device_slot();
  if (!smem_set[mode][dev]) {
    const cudaError_t e =
        mode == 0 ? cudaFuncSetAttribute(umma_attention_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM_BYTES)
        : mode == 1 ? cudaFuncSetAttribute(umma_attention_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM_BYTES)
                    : cudaFuncSetAttribute(umma_attention_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM_BYTES_ROT);
    if (e != cudaSuccess) return -1;
    smem_set[mode][dev] = true;
  }
  AttnArgs a{};
  a.items = items; a.cta_first = cta_first; a.row_pos = row_pos; a.out = out; a.page_table = page_table;
  a.rope = rope; a.rope_rows = rope_rows;
  a.partial_o = partial_o; a.partial_ml = partial_ml;
  a.n_q_heads = n_q_heads; a.n_kv_heads = n_kv_heads;
  a.scale_log2 = 1.4426950408889634f * 0.08838834764831845f;
  a.err_word = err_word;
  cudaError_t rc;
  if (mode == 1)
    rc = launch_pdl(umma_attention_kernel<1>, dim3(n_ctas), dim3(ATT_THREADS), ATT_SMEM_BYTES, s, maps.q, maps.k, maps.v, a);
  else if (mode == 2)
    rc = launch_pdl(umma_attention_kernel<2>, dim3(n_ctas), dim3(ATT_THREADS_ROT), ATT_SMEM_BYTES_ROT, s, maps.q, maps.k, maps.v, a);
  else
    rc = launch_pdl(umma_attention_kernel<0>, dim3(n_ctas), dim3(ATT_THREADS), ATT_SMEM_BYTES, s, maps.q, maps.k, maps.v, a);
  return rc == cudaSuccess ? 0 : -1;
}

}  // namespace pc
