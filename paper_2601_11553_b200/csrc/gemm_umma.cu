// Dense GEMM on the 5th-generation tensor cores: D[M][N] = A[M][K] * B[N][K]^T, fp16 operands,
// fp32 accumulation in TMEM, fused epilogues (QKV + RoPE + scatter, residual add, SwiGLU).
//
// One persistent CTA per SM, 320 threads, warp-specialised:
//   warp 0    TMA producer: one lane streams 128x64 A tiles and BNx64 B tiles (128-byte swizzle) into
//             a ring of shared-memory stages, signalling `full` mbarriers by transaction bytes;
//   warp 1    owns the TMEM allocation; one lane issues tcgen05.mma (128 x BN x 16) on each stage and
//             commits to the stage's `empty` barrier, then to the accumulator's `tmem_full` barrier;
//   warps 2-9 epilogue: each reads its 32-lane quarter of the accumulator with tcgen05.ld (two warps per
//             quarter, alternating 32-column chunks), applies the epilogue and stores; two accumulator
//             stages let the next tile's MMAs overlap it.
// Pair mode (PAIR = true): the grid is made of clusters of two CTAs on a 256 x BN tile.  Each CTA loads its own
// 128 rows of A and only half of the tile's B rows; the rank-0 CTA issues one cta_group::2 UMMA per K step that
// reads A and B from both shared memories and fills 128 TMEM lanes in each CTA, so the bytes a CTA pulls from
// L2 per MMA clock fall by a third (BN = 256) and the main loop stops being bound by that feed.  Barriers:
// `full` lives in rank 0 and counts both CTAs' TMA bytes; `empty` and `tmem_full` exist in both CTAs and are
// signalled together by a multicast commit; `tmem_empty` lives in rank 0 and collects both CTAs' epilogue warps.
// Every wait is bounded (ptx.cuh); on a timeout the roles fall through to the common teardown,
// the producer gives its outstanding copies time to land, TMEM is freed and the host sees the error word.
#include "epilogue.cuh"
#include "kernels.h"
#include "ptx.cuh"

namespace pc {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;                       // 64 fp16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int GEMM_THREADS = 320;               // TMA warp, MMA warp, 8 epilogue warps
constexpr int A_STAGE_BYTES = BM * BK * 2;   // 16 KB
// Epilogue staging: every epilogue warp owns two buffers of 32 rows x 64 bytes (pitch 80 to spread banks).
// A thread writes its accumulator row; the warp then reads the buffer back with four lanes per row, so that
// every global access of the epilogue (residual, RoPE table, outputs) has adjacent lanes on adjacent addresses.
constexpr int EPI_WARPS = 8;
constexpr int STG_PITCH = 80;
constexpr int STG_BUF_BYTES = 32 * STG_PITCH;
constexpr int EPI_STAGING_BYTES = EPI_WARPS * 2 * STG_BUF_BYTES;   // 40 KB

template <int BN, bool PAIR> struct GemmCfg {
  static constexpr int B_ROWS = PAIR ? BN / 2 : BN;                // rows of B this CTA loads per stage
  static constexpr int B_STAGE_BYTES = B_ROWS * BK * 2;
  static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
  static constexpr int STAGES = (B_ROWS >= 256) ? 3 : (B_ROWS >= 128 ? 5 : 6);
  static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
  static constexpr int SMEM_BYTES = RING_BYTES + EPI_STAGING_BYTES + 1024;   // + slack to align the ring to 1024 B
  static constexpr int TMEM_COLS = 2 * BN;                         // two accumulator stages
};

struct GemmArgs {
  int32_t M, N, K;
  int32_t k_splits;          // EPI_RESIDUAL only: the K range of a tile is cut into this many work items
  float* c;                  // EPI_STORE_F32
  QkvEpilogue qkv;           // EPI_QKV
  ResidualEpilogue res;      // EPI_RESIDUAL
  SwigluEpilogue swi;        // EPI_SWIGLU
  int* err_word;
};

template <int BN, int KIND, bool PAIR>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmArgs args) {
  using Cfg = GemmCfg<BN, PAIR>;
  constexpr int TILE_M = PAIR ? 2 * BM : BM;            // rows of a work item (both CTAs of a pair)
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;  // 0 issues the MMAs
  const int worker = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int n_workers = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int cta_failed;       // set by any role whose bounded wait ran out (or saw another role's error)

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  const int n_m_tiles = (args.M + TILE_M - 1) / TILE_M;
  const int n_n_tiles = args.N / BN;
  const int k_splits = (KIND == EPI_RESIDUAL) ? args.k_splits : 1;
  const int n_tiles = n_m_tiles * n_n_tiles * k_splits;      // work items: (tile, K part)
  const int n_kb_total = args.K / BK;
  // item -> (m tile, n tile, first and one-past-last 64-wide K block)
  auto kb_begin = [&](int item) { return ((item % k_splits) * n_kb_total) / k_splits; };
  auto kb_end = [&](int item) { return ((item % k_splits + 1) * n_kb_total) / k_splits; };

  if (threadIdx.x == 0) {
    cta_failed = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&tmem_full_bar[s], 1); mbar_init(&tmem_empty_bar[s], PAIR ? 16 : 8); }
    fence_mbar_init();
  }
  if (warp == 1) {
    if constexpr (PAIR) {
      tmem_alloc_pair<Cfg::TMEM_COLS>(&tmem_base_slot);
      tmem_relinquish_pair();
    } else {
      tmem_alloc<Cfg::TMEM_COLS>(&tmem_base_slot);
      tmem_relinquish();
    }
  }
  if (warp == 0 && lane == 0) {
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  pdl_launch_dependents();
  tc_fence_before_sync();
  __syncthreads();
  if constexpr (PAIR) {       // the other CTA's barriers must exist before anything is signalled there
    cluster_arrive();
    cluster_wait();
  }
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;
  // The A operand, the index arrays and the residual stream come from earlier kernels: nothing that touches them
  // runs before pdl_wait().  The weights do not, so the producer thread requests its first B tiles before it waits:
  // when this CTA starts while the previous kernel still runs on other SMs (programmatic launch), the first
  // DRAM round trip of the weights is over by the time the dependency resolves.
  const bool is_producer_thread = warp == 0 && lane == 0;
  if (!is_producer_thread) pdl_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // rank 0's barrier counts the bytes of both CTAs of a pair; each CTA loads its rows of A and its half of B
      auto expect = [&](int st) {
        if constexpr (PAIR) { if (rank == 0) mbar_arrive_expect_tx(&full_bar[st], 2 * Cfg::STAGE_BYTES); }
        else mbar_arrive_expect_tx(&full_bar[st], Cfg::STAGE_BYTES);
      };
      auto load_b = [&](int st, int kb, int n_idx) {
        uint8_t* b_dst = ring + st * Cfg::STAGE_BYTES + A_STAGE_BYTES;
        if constexpr (PAIR)
          tma_load_2d_pair(b_dst, &tmB, mapa_shared(smem_u32(&full_bar[st]), 0), kb * BK,
                           n_idx * BN + static_cast<int>(rank) * Cfg::B_ROWS);
        else tma_load_2d(b_dst, &tmB, &full_bar[st], kb * BK, n_idx * BN);
      };
      auto load_a = [&](int st, int kb, int m_idx) {
        uint8_t* a_dst = ring + st * Cfg::STAGE_BYTES;
        if constexpr (PAIR)
          tma_load_2d_pair(a_dst, &tmA, mapa_shared(smem_u32(&full_bar[st]), 0), kb * BK,
                           m_idx * TILE_M + static_cast<int>(rank) * BM);
        else tma_load_2d(a_dst, &tmA, &full_bar[st], kb * BK, m_idx * BM);
      };
      // weights of the first tile's first steps, into the still untouched stages
      int early = 0;
      if (worker < n_tiles) {
        const int n_idx = (worker / k_splits) % n_n_tiles;
        const int kb0 = kb_begin(worker);
        early = min(STAGES, kb_end(worker) - kb0);
        for (int i = 0; i < early; ++i) {
          expect(i);
          load_b(i, kb0 + i, n_idx);
        }
      }
      pdl_wait();
      for (int tile = worker; tile < n_tiles && ok; tile += n_workers) {
        const int m_idx = (tile / k_splits) / n_n_tiles, n_idx = (tile / k_splits) % n_n_tiles;
        for (int kb = kb_begin(tile); kb < kb_end(tile); ++kb) {
          if (early > 0) {            // this stage's barrier is armed and its B tile is on the way (or there)
            --early;
            load_a(stage, kb, m_idx);
          } else {
            if (!mbar_wait(&empty_bar[stage], phase ^ 1u, args.err_word, DEV_ERR_GEMM_PRODUCER)) { ok = false; cta_failed = 1; break; }
            expect(stage);
            load_a(stage, kb, m_idx);
            load_b(stage, kb, n_idx);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      (void)ok;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_f16(TILE_M, BN, /*fp16*/ 0, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = worker; tile < n_tiles && ok; tile += n_workers, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1u;
        if (!mbar_wait(&tmem_empty_bar[acc], acc_phase ^ 1u, args.err_word, DEV_ERR_GEMM_MMA)) { ok = false; cta_failed = 1; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        const int kb0 = kb_begin(tile), kb1 = kb_end(tile);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, args.err_word, DEV_ERR_GEMM_MMA)) { ok = false; cta_failed = 1; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(ring + stage * Cfg::STAGE_BYTES);
          const uint32_t b_addr = a_addr + A_STAGE_BYTES;
          const uint64_t a_desc = make_smem_desc_sw128(a_addr, 16, 1024);
          const uint64_t b_desc = make_smem_desc_sw128(b_addr, 16, 1024);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // 16 elements along K = 32 bytes = 2 units of the descriptor's 16-byte address field
            if constexpr (PAIR)
              umma_ss_pair(d_tmem, a_desc + static_cast<uint64_t>(2 * k), b_desc + static_cast<uint64_t>(2 * k), idesc,
                           (kb > kb0 || k != 0) ? 1u : 0u);
            else
              umma_ss(d_tmem, a_desc + static_cast<uint64_t>(2 * k), b_desc + static_cast<uint64_t>(2 * k), idesc,
                      (kb > kb0 || k != 0) ? 1u : 0u);
          }
          // stage reusable (in both CTAs of a pair) once these MMAs have read it
          if constexpr (PAIR) umma_commit_pair(&empty_bar[stage]); else umma_commit(&empty_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          if constexpr (PAIR) umma_commit_pair(&tmem_full_bar[acc]); else umma_commit(&tmem_full_bar[acc]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    // Two warps share every TMEM lane quarter and split the tile's columns between them.
    const int quarter = warp & 3;                 // TMEM lanes [32*quarter, 32*quarter + 32)
    const int cgroup = (warp - 2) >> 2;           // 0 or 1: which alternate 32-column chunks this warp takes
    uint8_t* stg = ring + Cfg::RING_BYTES + (warp - 2) * 2 * STG_BUF_BYTES;
    const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
    int it = 0;
    float4 nv0[4], nv1[4];       // EPI_RESIDUAL: residual values loaded ahead of the pass that consumes them
    // address of the four columns this lane handles in iteration `it4` of the pass starting at tile column c
    const uint32_t tmem_empty_remote = PAIR ? mapa_shared(smem_u32(&tmem_empty_bar[0]), 0) : 0u;
    auto res_ptr = [&](int m_idx, int n_idx, int c, int it4) {
      const int row = min(m_idx * BM + quarter * 32 + it4 * 8 + (lane >> 2), args.M - 1);
      return reinterpret_cast<float4*>(args.res.resid + static_cast<size_t>(row) * args.res.ld + n_idx * BN + c +
                                       (lane & 3) * 4);
    };
    for (int tile = worker; tile < n_tiles; tile += n_workers, ++it) {
      // m_idx counts 128-row blocks: this CTA's half of a pair's 256-row tile
      const int m_idx = ((tile / k_splits) / n_n_tiles) * (TILE_M / BM) + static_cast<int>(rank);
      const int n_idx = (tile / k_splits) % n_n_tiles;
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1u;
      if (KIND == EPI_RESIDUAL && k_splits == 1) {
        // the residual values of the tile's first pass travel while the main loop is still running
#pragma unroll
        for (int it = 0; it < 4; ++it) {
          float4* p0 = res_ptr(m_idx, n_idx, cgroup * 32, it);
          nv0[it] = p0[0];
          nv1[it] = p0[4];
        }
      }
      // EPI_QKV: everything the epilogue needs besides the accumulator depends on the tile alone, so it is
      // requested while the main loop still runs.  Every lane keeps the index entries of row (row_base + lane);
      // the four rows a lane stores in a pass (it * 8 + lane / 4) are fetched by shuffle.  The rotation depends on
      // the column inside a head, not on the head, so the two column groups a warp handles need two sets of table
      // entries per tile.
      QkvRow rws[4];
      RopeCs cs_all[2][4];
      if constexpr (KIND == EPI_QKV) {
        const QkvRow mine = load_qkv_row(args.qkv, min(m_idx * BM + quarter * 32 + lane, args.M - 1));
#pragma unroll
        for (int it4 = 0; it4 < 4; ++it4) {
          const int rl = it4 * 8 + (lane >> 2);
          rws[it4].pos = __shfl_sync(0xffffffffu, mine.pos, rl);
          rws[it4].slot = __shfl_sync(0xffffffffu, mine.slot, rl);
          rws[it4].pool_tok = __shfl_sync(0xffffffffu, mine.pool_tok, rl);
        }
#pragma unroll
        for (int p16 = 0; p16 < 2; ++p16)
#pragma unroll
          for (int it4 = 0; it4 < 4; ++it4)
            cs_all[p16][it4] = qkv_load_cs(args.qkv, rws[it4].pos, n_idx * (BN / HEAD_DIM),
                                           cgroup * 32 + p16 * 16 + (lane & 3) * 4);
      }
      bool ok = mbar_wait(&tmem_full_bar[acc], acc_phase, args.err_word, DEV_ERR_GEMM_EPILOGUE);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { cta_failed = 1; break; }
      tc_fence_after_sync();
      const uint32_t t_acc = tmem_base + lane_base + static_cast<uint32_t>(acc * BN);
      const int row_base = m_idx * BM + quarter * 32;          // first of this warp's 32 rows
      // Two 16-column groups per pass: `ca` and `cb` are tile columns; fn(rl, c4, valid, a, b) gets four
      // columns of each group (c4 = 0, 4, 8, 12) for local row rl, adjacent lanes on adjacent column groups.
      auto pass = [&](int ca, int cb, auto&& fn) {
        uint32_t ra[16], rb[16];
        tmem_ld_32x16(t_acc + ca, ra);
        tmem_ld_32x16(t_acc + cb, rb);
        tmem_wait_ld();
        uint4* wa = reinterpret_cast<uint4*>(stg + lane * STG_PITCH);
        uint4* wb = reinterpret_cast<uint4*>(stg + STG_BUF_BYTES + lane * STG_PITCH);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          wa[q] = make_uint4(ra[4 * q], ra[4 * q + 1], ra[4 * q + 2], ra[4 * q + 3]);
          wb[q] = make_uint4(rb[4 * q], rb[4 * q + 1], rb[4 * q + 2], rb[4 * q + 3]);
        }
        __syncwarp();
#pragma unroll
        for (int it = 0; it < 4; ++it) {
          const int rl = it * 8 + (lane >> 2);
          const float4 a = *reinterpret_cast<const float4*>(stg + rl * STG_PITCH + (lane & 3) * 16);
          const float4 b = *reinterpret_cast<const float4*>(stg + STG_BUF_BYTES + rl * STG_PITCH + (lane & 3) * 16);
          fn(rl, (lane & 3) * 4, row_base + rl < args.M, a, b);     // every lane calls fn (it may shuffle)
        }
        __syncwarp();
      };
      if constexpr (KIND == EPI_STORE_F32) {
#pragma unroll 1
        for (int c = cgroup * 32; c < BN; c += 64) {
          pass(c, c + 16, [&](int rl, int c4, bool valid, float4 a, float4 b) {
            if (!valid) return;
            float* dst = args.c + static_cast<size_t>(row_base + rl) * args.N + n_idx * BN + c + c4;
            *reinterpret_cast<float4*>(dst) = a;
            *reinterpret_cast<float4*>(dst + 16) = b;
          });
        }
      } else if (KIND == EPI_RESIDUAL && k_splits > 1) {
        // K is split over several work items: each adds its partial sums with vector atomics
        // (the order of the additions, hence the last bits, then depends on scheduling)
#pragma unroll 1
        for (int c = cgroup * 32; c < BN; c += 64) {
          pass(c, c + 16, [&](int rl, int c4, bool valid, float4 a, float4 b) {
            if (!valid) return;
            float4* dst = reinterpret_cast<float4*>(args.res.resid + static_cast<size_t>(row_base + rl) * args.res.ld +
                                                    n_idx * BN + c + c4);
            atomicAdd(dst, a);
            atomicAdd(dst + 4, b);
          });
        }
      } else if constexpr (KIND == EPI_RESIDUAL) {
        // read-modify-write of the fp32 residual stream.  The loads of a pass are issued one pass ahead
        // (those of the first pass before the accumulator is even waited for, see above) and all before the
        // stores they pair with: the compiler cannot move a load above a store to the same array by itself.
#pragma unroll 1
        for (int c = cgroup * 32; c < BN; c += 64) {
          float4 v0[4], v1[4];
#pragma unroll
          for (int it = 0; it < 4; ++it) { v0[it] = nv0[it]; v1[it] = nv1[it]; }
          float4* ptr[4];
#pragma unroll
          for (int it = 0; it < 4; ++it) {
            ptr[it] = res_ptr(m_idx, n_idx, c, it);
            if (c + 64 < BN) {                      // next pass of this tile
              float4* nx = res_ptr(m_idx, n_idx, c + 64, it);
              nv0[it] = nx[0];
              nv1[it] = nx[4];
            }
          }
          int it_ctr = 0;
          pass(c, c + 16, [&](int rl, int c4, bool valid, float4 a, float4 b) {
            (void)rl; (void)c4;
            const int it = it_ctr++;
            if (valid) {
              v0[it].x += a.x; v0[it].y += a.y; v0[it].z += a.z; v0[it].w += a.w;
              v1[it].x += b.x; v1[it].y += b.y; v1[it].z += b.z; v1[it].w += b.w;
              ptr[it][0] = v0[it];
              ptr[it][4] = v1[it];
            }
          });
        }
      } else if constexpr (KIND == EPI_QKV) {
#pragma unroll 1
        for (int hl = 0; hl < BN / HEAD_DIM; ++hl) {
          const int hb = n_idx * (BN / HEAD_DIM) + hl;
#pragma unroll
          for (int p16 = 0; p16 < 2; ++p16) {
            const int c0 = cgroup * 32 + p16 * 16;                       // low-half column of this pass
            int it_ctr = 0;
            pass(hl * HEAD_DIM + c0, hl * HEAD_DIM + ROPE_HALF + c0, [&](int rl, int c4, bool valid, float4 lo, float4 hi) {
              const int it4 = it_ctr++;
              if (valid) qkv_store4_cs(args.qkv, row_base + rl, rws[it4], hb, c0 + c4, lo, hi, cs_all[p16][it4]);
            });
          }
        }
      } else {   // EPI_SWIGLU: every 128-column block holds 64 gate columns, then the matching 64 up columns
        // A thread has gate and up of the same (row, column) in hand as they come from TMEM, so silu(g) * u is
        // formed and rounded to fp16 first and only the result crosses shared memory: 32 bytes per row instead of
        // 128 (the staging competes with the MMA's operand reads for shared-memory bandwidth and was the largest
        // part of this epilogue).
        // The way through shared memory has a long latency while the MMA is reading operands, so the passes are
        // software-pipelined over the warp's two staging buffers: pass p is written, then pass p - 1 (written one
        // step earlier) is read back and stored.
        constexpr int PITCH = 48;               // 32 bytes of a row + 16: lanes land on distinct 16-byte slots
        constexpr int N_PASS = 2 * (BN / 128);
        auto out_col = [&](int p) { return (n_idx * (BN / 128) + (p >> 1)) * 64 + cgroup * 32 + (p & 1) * 16; };
        auto drain = [&](int p) {               // read pass p back, four lanes per row, and store it
          const uint8_t* buf = stg + (p & 1) * STG_BUF_BYTES;
#pragma unroll
          for (int it = 0; it < 4; ++it) {
            const int rl = it * 8 + (lane >> 2);
            const uint2 v = *reinterpret_cast<const uint2*>(buf + rl * PITCH + (lane & 3) * 8);
            if (row_base + rl < args.M)
              *reinterpret_cast<uint2*>(args.swi.act + static_cast<size_t>(row_base + rl) * args.swi.ld + out_col(p) +
                                        (lane & 3) * 4) = v;
          }
        };
#pragma unroll
        for (int p = 0; p < N_PASS; ++p) {
          const int c0 = (p >> 1) * 128 + cgroup * 32 + (p & 1) * 16;
          uint32_t rg[16], ru[16];
          tmem_ld_32x16(t_acc + c0, rg);
          tmem_ld_32x16(t_acc + 64 + c0, ru);
          tmem_wait_ld();
          uint32_t o[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            o[i] = pack_half2(silu_f(__uint_as_float(rg[2 * i])) * __uint_as_float(ru[2 * i]),
                              silu_f(__uint_as_float(rg[2 * i + 1])) * __uint_as_float(ru[2 * i + 1]));
          uint4* w = reinterpret_cast<uint4*>(stg + (p & 1) * STG_BUF_BYTES + lane * PITCH);
          w[0] = make_uint4(o[0], o[1], o[2], o[3]);
          w[1] = make_uint4(o[4], o[5], o[6], o[7]);
          __syncwarp();                          // pass p is visible to the whole warp
          if (p > 0) {
            drain(p - 1);
            __syncwarp();                        // all lanes have read that buffer before pass p + 1 rewrites it
          }
        }
        drain(N_PASS - 1);
        __syncwarp();
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if constexpr (PAIR) mbar_arrive_cluster(tmem_empty_remote + static_cast<uint32_t>(acc) * 8u);
        else mbar_arrive(&tmem_empty_bar[acc]);
      }
    }
  }

  // ------------------------------------------------------------------ teardown (every thread gets here)
  tc_fence_before_sync();
  __syncthreads();
  if (cta_failed) {
    // Error path only (the flag was written before the barrier, so every thread takes the same branch): whichever
    // role gave up, bulk copies this CTA issued may still be on their way into its shared memory; give them time to
    // land before the memory is released.
    if (threadIdx.x == 0) {
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < DRAIN_LIMIT_NS) { }
    }
    __syncthreads();
  }
  if constexpr (PAIR) {       // neither CTA may leave while the other can still read its memory or signal it
    cluster_arrive();
    cluster_wait();
  }
  if (warp == 1) {
    tc_fence_after_sync();
    if constexpr (PAIR) tmem_dealloc_pair<Cfg::TMEM_COLS>(tmem_base);
    else tmem_dealloc<Cfg::TMEM_COLS>(tmem_base);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

template <int BN, int KIND, bool PAIR>
int launch_one(const GemmOperand& A, const GemmOperand& B, const GemmArgs& args, int n_sms, cudaStream_t s) {
  using Cfg = GemmCfg<BN, PAIR>;
  static bool smem_set[MAX_DEVICES] = {};      // per kernel instantiation and device
  const int dev = current_device_slot();
  if (!smem_set[dev]) {
    if (cudaFuncSetAttribute(umma_gemm_kernel<BN, KIND, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::SMEM_BYTES) != cudaSuccess)
      return -1;
    smem_set[dev] = true;
  }
  constexpr int TILE_M = PAIR ? 2 * BM : BM;
  const int n_tiles = ((args.M + TILE_M - 1) / TILE_M) * (args.N / BN) * (args.k_splits > 0 ? args.k_splits : 1);
  if (n_tiles <= 0) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(GEMM_THREADS);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int workers = n_sms;
  if (PAIR) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
    // SMs pair up inside a GPC only, so fewer than n_sms / 2 clusters may be resident at once; a persistent
    // grid larger than that would run its last clusters after all the others
    static int max_clusters_of[MAX_DEVICES] = {};      // per kernel instantiation and device
    int& max_clusters = max_clusters_of[dev];
    if (max_clusters == 0) {
      cfg.gridDim = dim3((n_sms / 2) * 2);
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, umma_gemm_kernel<BN, KIND, PAIR>, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return -1;
      }
      max_clusters = n;
    }
    workers = max_clusters < n_sms / 2 ? max_clusters : n_sms / 2;
  }
  cfg.gridDim = dim3((n_tiles < workers ? n_tiles : workers) * (PAIR ? 2 : 1));
  return cudaLaunchKernelEx(&cfg, umma_gemm_kernel<BN, KIND, PAIR>, A.map, B.map, args) == cudaSuccess ? 0 : -1;
}

}  // namespace

int init_driver_api() {
  if (g_encode) return 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess) return -1;
  if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return -1;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return 0;
}

int encode_f16_map(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                   const uint32_t* box) {
  if (init_driver_api() != 0) return -1;
  cuuint64_t gdim[5];
  cuuint64_t gstr[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  const CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, static_cast<cuuint32_t>(rank),
                              const_cast<void*>(base), gdim, gstr, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -1;
}

int make_operand_map(GemmOperand* out, const void* base, int64_t rows, int64_t cols, int box_rows) {
  const uint64_t dims[2] = {static_cast<uint64_t>(cols), static_cast<uint64_t>(rows)};
  const uint64_t strides[1] = {static_cast<uint64_t>(cols) * 2};
  const uint32_t box[2] = {static_cast<uint32_t>(BK), static_cast<uint32_t>(box_rows)};
  return encode_f16_map(&out->map, base, 2, dims, strides, box);
}

// Tile shape (and, for the residual GEMMs, the number of K parts) for a problem.  The main loop of a single
// CTA is fed at roughly 64 bytes per clock from L2, so a 128 x 128 x 64 step (32 KB) costs about 512 clocks and
// a 128 x 256 x 64 step (48 KB) about 768; a CTA pair on a 256 x 256 tile loads 32 KB per CTA and step and its
// step costs about 600 clocks.  A work item also pays about three steps of ramp-up and tail.  The cost of a
// choice is (rounds of items over the workers) x (steps per item + 3) x (clocks per step).
// Measured on B200 (M = 33 024, d = 1024), single CTAs -> pairs: O-projection 990 -> 1183 TFLOP/s (K = 2048), down-
// projection 1059 -> 1280 (K = 3072), and, once their epilogues had been shortened, QKV 1103 -> 1149 and gate/up
// 1269 -> 1392 (K = 1024); at M = 2176, d = 2048: QKV 886 -> 966, gate/up 1037 -> 1213.  At M = 1344 pairs made the
// whole step 0.8 % slower (three runs each), hence the thresholds below.
void umma_gemm_pick_shape(int M, int N, int K, int n_sms, bool may_split_k, bool may_pair, int* block_n,
                          int* k_splits, int* pair) {
  const int n_kb = K / BK;
  int64_t best = INT64_MAX;
  *block_n = 128;
  *k_splits = 1;
  *pair = 0;
  for (int shape = 0; shape < 3; ++shape) {           // 128 x 128, 128 x 256, pair 256 x 256
    const int bn = shape == 0 ? 128 : 256;
    const bool pr = shape == 2;
    if (N % bn != 0 || (pr && (!may_pair || n_sms < 2))) continue;
    const int tile_m = pr ? 2 * BM : BM;
    const int workers = pr ? n_sms / 2 : n_sms;
    const int64_t clocks = shape == 0 ? 512 : (shape == 1 ? 768 : 600);
    const int64_t tiles = static_cast<int64_t>((M + tile_m - 1) / tile_m) * (N / bn);
    // small problems are bound by ramp-up and tail, which pairs lengthen: the residual GEMMs (long K) take pairs
    // from half a round of pair tiles, the others (K = d_model, epilogue-heavy) from one and a half rounds
    if (pr && tiles * 2 < (may_split_k ? 1 : 3) * workers) continue;
    for (int sp = 1; sp <= (may_split_k ? 8 : 1); ++sp) {
      if (sp > 1 && n_kb / sp < 4) break;
      const int64_t rounds = (tiles * sp + workers - 1) / workers;
      const int64_t cost = rounds * ((n_kb + sp - 1) / sp + 3) * clocks;
      // prefer later shapes and fewer parts on ties; a split must win by 10 %
      const bool better = sp == 1 ? cost <= best : cost * 10 < best * 9;
      if (better) { best = cost; *block_n = bn; *k_splits = sp; *pair = pr ? 1 : 0; }
    }
  }
}
template <int BN, bool PAIR>
static int launch_bn(const GemmOperand& A, const GemmOperand& B, GemmArgs& args, GemmEpilogueKind kind,
                     const void* epilogue, int n_sms, cudaStream_t s) {
  switch (kind) {
    case EPI_STORE_F32:
      return launch_one<BN, EPI_STORE_F32, PAIR>(A, B, args, n_sms, s);
    case EPI_QKV:
      args.qkv = *static_cast<const QkvEpilogue*>(epilogue);
      return launch_one<BN, EPI_QKV, PAIR>(A, B, args, n_sms, s);
    case EPI_RESIDUAL:
      args.res = *static_cast<const ResidualEpilogue*>(epilogue);
      return launch_one<BN, EPI_RESIDUAL, PAIR>(A, B, args, n_sms, s);
    case EPI_SWIGLU:
      args.swi = *static_cast<const SwigluEpilogue*>(epilogue);
      return launch_one<BN, EPI_SWIGLU, PAIR>(A, B, args, n_sms, s);
  }
  return -1;
}

int launch_umma_gemm(const GemmOperand& A, const GemmOperand& B, int M, int N, int K, int block_n,
                     GemmEpilogueKind kind, const void* epilogue, float* c_f32, int* err_word, int n_sms,
                     cudaStream_t s, int k_splits, int pair) {
  if (M <= 0) return 0;
  if (K % BK != 0 || N % block_n != 0 || (block_n != 128 && block_n != 256)) return -1;
  if (k_splits < 1 || (k_splits > 1 && kind != EPI_RESIDUAL) || k_splits > K / BK) return -1;
  if (pair && (block_n != 256 || n_sms < 2)) return -1;
  GemmArgs args{};
  args.M = M; args.N = N; args.K = K; args.c = c_f32; args.err_word = err_word; args.k_splits = k_splits;
  if (pair) return launch_bn<256, true>(A, B, args, kind, epilogue, n_sms, s);
  return block_n == 256 ? launch_bn<256, false>(A, B, args, kind, epilogue, n_sms, s)
                        : launch_bn<128, false>(A, B, args, kind, epilogue, n_sms, s);
}

}  // namespace pc
