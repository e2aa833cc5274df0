// Internal interface between the host runtime and the CUDA kernels (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

namespace pc {

constexpr int PAGE_TOKENS = 16;
constexpr int HEAD_DIM = 128;
constexpr int ROPE_HALF = HEAD_DIM / 2;

// One unit of gather work: up to 16 consecutive tokens of one stored page go to consecutive
// context slots of one prompt.  `pos` is the position (slot inside the prompt) of the first token.
struct GatherItem {
  int32_t dst_slot;   // global context slot (prompts of a batch are laid out back to back)
  int32_t src_page;   // page of the store
  int32_t n_tok;      // 1..16
  int32_t pos;        // RoPE position of the first token
};

// Per new row (device arrays of length M).
struct RowIndex {
  const int32_t* slot;      // global context slot of the row
  const int32_t* pos;       // position inside its prompt
  const int32_t* pool_tok;  // page * 16 + offset where the row's unrotated K/V is kept, or -1
};

// Attention work item: up to 128 consecutive new rows of one prompt (a tile), one unit (KV head g and
// pair of its query heads: unit = g * pairs + pair), against the context blocks [blk_begin, blk_end)
// (128 slots each).  The host deals items to the persistent CTAs so that each gets the same number of
// blocks; a unit whose blocks end up in several items is "split": each part writes an unnormalised
// partial result to its own slot and a second kernel merges the parts.
struct AttnItem {
  int32_t row0;          // first new row (global row index)
  int32_t n_rows;        // 1..128
  int32_t ctx0;          // global context slot of the prompt's slot 0
  int32_t blk_begin;     // first context block of this item
  int32_t blk_end;       // one past its last block
  int32_t partial_slot;  // -1: the item covers the unit's whole context and writes the final rows
  int32_t unit;
  int32_t pad0;
};

// Merge of the parts of one split unit: part s is in slot partial_slot0 + s.
struct AttnMerge {
  int32_t row0, n_rows;
  int32_t partial_slot0, n_parts;
  int32_t unit;
  int32_t pad0, pad1, pad2;
};

// Decode-step attention (attn_decode.cu): one block per (row, KV head, chunk of context slots).
struct DecodeAttnItem {
  int32_t row;           // new row (= prompt index in a decode step)
  int32_t ctx0;          // global context slot of the prompt's slot 0
  int32_t slot_begin;    // first slot of the chunk (slot inside the prompt)
  int32_t slot_end;      // one past its last slot (at most position + 1)
  int32_t kv_head;
  int32_t partial_slot;  // where the chunk's unnormalised result goes
  int32_t pad0, pad1;
};
struct DecodeAttnMerge {   // the chunks of one (row, KV head) are in slots partial_slot0 .. + n_parts - 1
  int32_t row, kv_head, partial_slot0, n_parts;
  int32_t pad0, pad1, pad2, pad3;
};
// partial_o: fp32 [items][query heads per KV head][128]; partial_ml: fp32 [items][query heads per KV head][2].
// Query heads per KV head must be 2 or 4.
// page_table != nullptr: the paged form (after a gather-free prefill): K and V are read from the bf16 pages of the
// layer through the page table, K rotated on load with the (cos, sin) table; an item's ctx0 then indexes its prompt's
// first page-table entry and kctx_layer / vctx_layer are unused.
int launch_decode_attention(const DecodeAttnItem* items, int n_items, const DecodeAttnMerge* merges, int n_merges,
                            const __half* q, const __half* kctx_layer, const __half* vctx_layer, float* partial_o,
                            float* partial_ml, __half* out, int n_q_heads, int n_kv_heads, cudaStream_t s,
                            const __nv_bfloat16* kpool_layer = nullptr, const __nv_bfloat16* vpool_layer = nullptr,
                            const int32_t* page_table = nullptr, const float2* rope = nullptr);

// A tile before scheduling: its rows and the number of 128-slot context blocks its last row can see.
struct AttnBaseTile { int32_t row0, n_rows, ctx0, n_blocks; };
// Deals (tile, unit, block range) items to at most n_sms CTAs (attn_plan.cu).  cta_first gets one entry per
// CTA used plus one; returns the plan's estimated makespan in quarter blocks.
int64_t plan_attention(const std::vector<AttnBaseTile>& tiles, int units_per_tile, int n_sms, int max_partial_slots,
                       std::vector<AttnItem>* items, std::vector<int32_t>* cta_first, std::vector<AttnMerge>* merges);

struct ModelDims {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, d_ffn;
  int32_t q_dim, kv_dim, qkv_dim;
  float rms_eps;
};

// ---- element-wise and memory-bound kernels (kernels_mem.cu)
void launch_build_rope_table(float2* table, int max_pos, double theta, cudaStream_t s);
void launch_bf16_to_f16(const __nv_bfloat16* src, __half* dst, int64_t n, cudaStream_t s);
// dst[(2*b + which) * blk + r][:] = src_which[b * blk + r][:]  (gate/up row interleave in blocks of blk rows)
void launch_interleave_rows_bf16_to_f16(const __nv_bfloat16* gate, const __nv_bfloat16* up, __half* dst, int rows,
                                        int cols, int blk, cudaStream_t s);
void launch_bf16_to_f32(const __nv_bfloat16* src, float* dst, int64_t n, cudaStream_t s);
// out row r = norm of x row (row_index ? row_index[r] : r); row_index is host-written before the call's first kernel
void launch_rmsnorm(const float* x, const float* gain, __half* out, int M, int d, float eps, cudaStream_t s,
                    const int32_t* row_index = nullptr);
void launch_gather_rerope(const GatherItem* items, int n_items, int n_layers, const __nv_bfloat16* kpool,
                          const __nv_bfloat16* vpool, int64_t pool_pages, __half* kctx, __half* vctx,
                          int64_t ctx_cap, int kv_dim, const float2* rope, cudaStream_t s);
// chunk [L][n][kv_dim] <-> pages (to_pool = 1: chunk -> pool)
void launch_chunk_pages_copy(__nv_bfloat16* chunk, __nv_bfloat16* pool, const int32_t* pages, int n_tokens,
                             int n_layers, int64_t pool_pages, int kv_dim, int to_pool, cudaStream_t s);
void launch_fill_synthetic(__nv_bfloat16* kpool, __nv_bfloat16* vpool, const int32_t* pages, int n_tokens,
                           int n_layers, int64_t pool_pages, int kv_dim, uint64_t seed, uint64_t chunk_id,
                           cudaStream_t s);

// ---- epilogue parameter blocks shared by the reference and the tcgen05 GEMMs
struct QkvEpilogue {
  RowIndex rows;
  const float2* rope;
  __half* q_out;              // [M][q_dim]
  __nv_bfloat16* kpool;       // layer base: [pool_pages*16][kv_dim]
  __nv_bfloat16* vpool;
  __half* kctx;               // layer base: [ctx_cap][kv_dim]
  __half* vctx;
  int32_t n_q_heads, n_kv_heads;
  // Paper-faithful mode: every row owns a page slot (rows.pool_tok >= 0) and Q, K, V all go to pages as bf16, Q and K
  // after rotation (what the attention uses and what the cache then holds); q_out, kctx, vctx are unused.
  __nv_bfloat16* qpool;       // layer base: [pool_pages*16][q_dim], or nullptr outside that mode
  int32_t paged;
  // Gather-free form of the default mode: the attention reads K and V from the pages, so nothing is written to the
  // assembled context (every row then has a page slot).
  int32_t skip_ctx;
};
struct ResidualEpilogue { float* resid; int32_t ld; };          // resid[row][col] += acc
struct SwigluEpilogue { __half* act; int32_t ld; };             // act[row][j] = silu(gate) * up

// ---- plain reference kernels (kernels_ref.cu)
void launch_ref_gemm(const __half* A, const __half* B, float* C, int M, int N, int K, cudaStream_t s);
void launch_ref_qkv_epilogue(const float* C, int M, const QkvEpilogue& e, cudaStream_t s);
void launch_ref_residual_epilogue(const float* C, int M, int N, const ResidualEpilogue& e, cudaStream_t s);
void launch_ref_swiglu_epilogue(const float* C, int M, int F, int blk, const SwigluEpilogue& e, cudaStream_t s);
void launch_ref_attention(const __half* q, const __half* kctx, const __half* vctx, __half* out, const int32_t* row_pos,
                          const int32_t* row_ctx0, int M, int n_q_heads, int n_kv_heads, cudaStream_t s);

// ---- tcgen05 GEMM (gemm_umma.cu).  A [M][K] fp16 row-major, B [N][K] fp16 row-major, D = A * B^T.
enum GemmEpilogueKind { EPI_STORE_F32 = 0, EPI_QKV = 1, EPI_RESIDUAL = 2, EPI_SWIGLU = 3 };
struct GemmOperand {           // a tensor map made once for a fixed buffer
  CUtensorMap map;
};
// rows x cols fp16 row-major matrix; box = box_rows x 64 columns, 128-byte swizzle
int make_operand_map(GemmOperand* out, const void* base, int64_t rows, int64_t cols, int box_rows);
// pair = 1 (block_n 256 only): clusters of two CTAs on 256 x 256 tiles; B's map then has box_rows = 128.
int launch_umma_gemm(const GemmOperand& A, const GemmOperand& B, int M, int N, int K, int block_n,
                     GemmEpilogueKind kind, const void* epilogue, float* c_f32, int* err_word, int n_sms,
                     cudaStream_t s, int k_splits = 1, int pair = 0);
constexpr int UMMA_GEMM_MIN_BLOCK_N = 128;       // narrowest N tile (a B operand map needs box_rows = the tile used)
// tile width, number of K parts (parts > 1 only if may_split_k: the residual epilogue then adds atomically) and
// whether CTA pairs are used (only if may_pair)
void umma_gemm_pick_shape(int M, int N, int K, int n_sms, bool may_split_k, bool may_pair, int* block_n,
                          int* k_splits, int* pair);

// ---- projections for at most SMALL_GEMM_MAX_ROWS rows on the CUDA cores, bound by reading W once (gemm_small.cu).
// D[M][N] = A[M][K] * W[N][K]^T with the epilogue `kind` (EPI_QKV, EPI_RESIDUAL or EPI_SWIGLU, parameter block as
// for the tcgen05 GEMM).  Input: x_f32 + gain (the RMSNorm of fp32 rows is applied on the way; QKV and SwiGLU) or
// a_f16 (residual kind).  gu_blk: gate / up row interleave of W for EPI_SWIGLU.  K % 256 == 0.
constexpr int SMALL_GEMM_MAX_ROWS = 8;
int launch_small_gemm(GemmEpilogueKind kind, const void* epilogue, int M, int N, int K, const float* x_f32,
                      const float* gain, float eps, const __half* a_f16, const __half* w, int gu_blk, int n_sms,
                      cudaStream_t s);

// rank-N fp16 tensor map with 128-byte swizzle; dims/strides innermost first (strides in bytes, from dim 1)
int encode_f16_map(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                   const uint32_t* box);

// ---- tcgen05 attention (attn_umma.cu)
struct AttnMaps { CUtensorMap q, k, v; };
int make_attn_maps(AttnMaps* out, const __half* q, int64_t m_cap, int q_dim, const __half* kctx_layer,
                   const __half* vctx_layer, int64_t ctx_cap, int kv_dim);
// partial_o: fp32 [slots][2 heads][128 rows][128]; partial_ml: fp32 [slots][2][128][2] (reference max, sum).
// CTA c (of n_ctas) runs items [cta_first[c], cta_first[c + 1]).
// mode 0: Q from the query buffer, K/V from the assembled context (maps over those buffers).
// mode 1: Q, K, V from the pages (maps from make_paged_attn_maps; paper-faithful mode).
// mode 2: Q from the query buffer (maps.q), K and V from the pages (maps.k, maps.v: one 16-row page per copy); K is
//         staged unrotated and rotated on its way to the MMA with the (cos, sin) table `rope` of rope_rows positions.
// In modes 1 and 2 an item's ctx0 is the index of its prompt's first entry in page_table.
int launch_umma_attention(const AttnMaps& maps, const AttnItem* items, const int32_t* cta_first, int n_ctas,
                          const int32_t* row_pos, __half* out, float* partial_o, float* partial_ml, int n_q_heads,
                          int n_kv_heads, int* err_word, cudaStream_t s, const int32_t* page_table = nullptr,
                          int mode = 0, const float2* rope = nullptr, int rope_rows = 0);
// Maps for the paged form of the attention (paper-faithful mode): Q, K and V are read straight from the bf16 pages
// of one layer, 16 rows (one page) per bulk copy; an item's ctx0 then is the index of its prompt's first entry in
// page_table (one page id per 16 context slots, padded to whole 128-slot blocks).
int make_paged_attn_maps(AttnMaps* out, const __nv_bfloat16* qpool_layer, const __nv_bfloat16* kpool_layer,
                         const __nv_bfloat16* vpool_layer, int64_t pool_pages, int q_dim, int kv_dim);
void launch_attention_merge(const AttnMerge* merges, int n_merges, const float* partial_o, const float* partial_ml,
                            __half* out, int n_q_heads, int n_kv_heads, cudaStream_t s);

int init_driver_api();   // resolves cuTensorMapEncodeTiled once; 0 on success

// Kernel attributes (dynamic shared memory limit) and cluster occupancy belong to a device, not to the process:
// launch helpers remember what they have set per device ordinal.
constexpr int MAX_DEVICES = 64;
inline int current_device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return 0;
  return dev;
}

// Launch with programmatic stream serialisation (see pdl_wait() in ptx.cuh).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

}  // namespace pc
