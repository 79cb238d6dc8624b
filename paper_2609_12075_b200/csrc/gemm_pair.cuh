// The projection kernel for large token counts: two-SM products (tcgen05 cta_group::2).
//
// Same orientation and epilogues as gemm_tc_kernel (weights = the M side, tokens = the N side, accumulator lane =
// feature, column = token), but a tile belongs to a pair of blocks (a cluster of two, one block per SM): the pair
// multiplies 256 output features by `tile_tok` tokens (any multiple of 16 up to 256).  Each block brings in its own
// 128 weight rows (256 for a gate/up pair: 128 gate rows, 128 up rows) and ONE HALF of the token tile - the even
// block the first half - with ordinary TMA copies; the product reads the other half out of the partner's shared
// memory.  Shared memory moves 128 bytes per cycle and has to carry the incoming stage plus the operand reads of
// every product, which bounds a one-SM 128-token tile at about half of the tensor peak; halving the token operand's
// share lifts that bound (256-token tiles become product-bound).
//
// Hand-overs: the ring's "stage filled" barriers live in the even block, which also issues the products; every copy
// of either block reports its bytes there (the copy's cta_group::2 form lets it name the partner's barrier).  "Stage
// free" and "accumulator complete" are signalled to both blocks by the product pipe (one tcgen05.commit per block, the
// partner's barrier named by its cluster address).  "Accumulator drained" is counted in the even block: the odd block's
// epilogue warps arrive remotely.  Every wait is bounded; a block that gave up raises the status word.
//
// Warp roles per block (256 threads): warp 0 = weight copies, warp 6 = token copies, warp 1 = tensor-memory
// allocation (+ product issue in the even block), warps 2..5 = epilogue.  The sum over k is one chain in k order,
// whatever the grid: results do not depend on the SM budget.
//
// The three single threads that drive the ring (two copy issuers, one product issuer) have nothing to hide their own
// instruction latencies behind; measured on B200, a barrier test costs such a thread about 160 cycles, a commit 70, a
// product 50-60, whatever the tile.  Each of them therefore tests the barrier of its NEXT stage inside the same
// instruction sequence that issues the current stage's work (ptx::umma_step_*, ptx::tma_load_2d_pair_step), keeps
// barrier addresses and descriptor halves in 32-bit registers, and polls without a clock read.
#pragma once
#include "gemm_tc.cuh"

namespace adit {
namespace tc {

template <bool DUAL, int EPI, int CW, bool INSTR>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a, GemmArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];   // used in the even block only
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t acc_full_bar[2];
  __shared__ __align__(8) uint64_t acc_empty_bar[2];       // used in the even block only
  __shared__ uint32_t tmem_base_smem;
  __shared__ volatile int abort_flag;
  __shared__ float red[4 * 256];
  __shared__ float rs_tile[256];

  ptx::pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned long long* const trace = INSTR ? g.trace : nullptr;
  // optional phase stamps (test aid): 0 start, 1 set-up done, 2 first / 3 last k-block issued, 4 accumulator seen
  // complete, 5 epilogue done, 6 end (12, 13: the SM's cycle counter at 0 and 6)
  unsigned long long* const dbg = (INSTR && g.dbg) ? g.dbg + (size_t)blockIdx.x * 16 : nullptr;
  if (dbg && threadIdx.x == 0) { dbg[0] = ptx::globaltimer_ns(); dbg[12] = (unsigned long long)clock64(); }
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4] = ptx::globaltimer_ns();
  uint8_t* tiles = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  constexpr int NV = DUAL ? 2 : 1;
  const int rank = (int)ptx::cluster_ctarank();  // 0 = even block of the pair (issues the products)
  const int half = g.tile_tok / 2;               // tokens of a tile that this block brings in
  const uint32_t w_bytes = NV * TILE_F * TILE_K * 2;
  const uint32_t a_bytes = (uint32_t)half * TILE_K * 2;
  const uint32_t stage_bytes = w_bytes + a_bytes;
  const int n_pairs = gridDim.x >> 1, pid = blockIdx.x >> 1;
  const int n_fpairs = (g.n_ftiles + 1) >> 1;
  const int total_items = n_fpairs * g.n_ttiles;
  const int acc_cols = NV * g.tile_tok;
  const int kbn = g.kb_total;

  if (threadIdx.x == 0) {
    for (int s = 0; s < g.stages; ++s) {
      ptx::mbar_init(&full_bar[s], 1);  // the even block's weight producer announces the bytes of both blocks
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&acc_full_bar[a], 1);
      ptx::mbar_init(&acc_empty_bar[a], 8);  // the four epilogue warps of either block
    }
    abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_w);
    ptx::prefetch_tensormap(&map_a);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(&tmem_base_smem, g.tmem_cols);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  // both blocks have initialised their barriers and hold their tensor memory before either signals the other
  ptx::cluster_arrive_release();
  ptx::cluster_wait_acquire();
  ptx::tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  if (dbg && threadIdx.x == 0) dbg[1] = ptx::globaltimer_ns();

  if (warp == 0 || warp == 6) {
    // ------------------------------ TMA producers ------------------------------
    const bool is_w = warp == 0;
    if (lane == 0) {
      const uint32_t full0 = ptx::mapa_shared(ptx::smem_u32(&full_bar[0]), 0);  // the even block's barriers
      int pre = 0;
      if (pid < total_items) {
        // weights do not depend on the preceding kernel: as many blocks as the ring holds are requested at once
        const int ft = (pid % n_fpairs) * 2 + rank;
        pre = min(kbn, g.stages);
        if (is_w)
          for (int i = 0; i < pre; ++i) {
            if (rank == 0) ptx::mbar_arrive_expect_tx(&full_bar[i], 2 * stage_bytes);
            ptx::tma_load_2d_pair(tiles + (size_t)i * stage_bytes, &map_w, i * TILE_K, ft * NV * TILE_F, full0 + 8u * i);
          }
      }
      ptx::pdl_wait_prior_grids();
      if (trace && is_w) trace[blockIdx.x * 4 + 1] = ptx::globaltimer_ns();
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      bool ready = false;  // the next stage is known to be free (tested one step ahead)
      for (int w = pid; w < total_items && ok; w += n_pairs) {
        const int ft = (w % n_fpairs) * 2 + rank, tt = w / n_fpairs;
        const int w_row = ft * NV * TILE_F, a_row = tt * g.tile_tok + rank * half;
        for (int kb = 0; kb < kbn; ++kb, ++issued) {
          uint8_t* ws = tiles + (size_t)stage * stage_bytes;
          if (issued >= pre && !ready && !ptx::mbar_wait_hot(&empty_bar[stage], phase ^ 1)) { ok = false; break; }
          const int cur = stage;
          if (++stage == g.stages) { stage = 0; phase ^= 1; }
          // (the stages requested ahead of the dependency wait have never been used: nothing to test for them)
          uint64_t* const next_free = &empty_bar[stage];
          if (is_w) {
            if (issued >= pre)
              ready = ptx::tma_load_2d_pair_step(ws, &map_w, kb * TILE_K, w_row, full0 + 8u * cur, &full_bar[cur],
                                                 rank == 0 ? 2 * stage_bytes : 0u, next_free, phase ^ 1);
            else
              ready = issued + 1 >= pre && ptx::mbar_test_wait(next_free, phase ^ 1);
          } else {
            ready = ptx::tma_load_2d_pair_step(ws + w_bytes, &map_a, kb * TILE_K, a_row, full0 + 8u * cur, &full_bar[cur], 0u, next_free,
                                               phase ^ 1);
          }
        }
      }
      if (!ok) { atomicExch(g.status, -6); abort_flag = 1; }
    }
  } else if (warp == 1) {
    // ------------------------------ product issue (even block) ------------------------------
    if (lane == 0 && rank == 0) {
      // This thread has nothing to hide its own instruction latencies behind, and a k-block's products have to leave
      // it every few hundred cycles: everything it touches per k-block is a 32-bit register (shared-memory addresses of
      // the barriers, low descriptor halves), advanced with one add per stage.
      const uint32_t idesc = ptx::idesc_bf16_f32(2 * TILE_F, g.tile_tok);
      const uint32_t hi = ptx::smem_desc_hi_sw128();
      const uint32_t w_lo0 = ptx::smem_desc_lo(ptx::smem_u32(tiles)), a_lo0 = ptx::smem_desc_lo(ptx::smem_u32(tiles) + w_bytes);
      const uint32_t lo_step = stage_bytes >> 4;
      const uint32_t full0 = ptx::smem_u32(&full_bar[0]), empty0 = ptx::smem_u32(&empty_bar[0]);
      const uint32_t bar_end = 8u * (uint32_t)g.stages;  // byte offset one past the last stage's barrier
      const uint32_t d2_off = (uint32_t)g.tile_tok, up_lo = TILE_F * TILE_K * 2 >> 4;
      uint32_t boff = 0, phase = 0, w_lo = w_lo0, a_lo = a_lo0;  // current stage: barrier byte offset, parity, descriptors
      int acc_iter = 0;
      bool ok = true;
      bool ready = false;  // the next k-block's stage is known to be filled (tested one step ahead)
      for (int w = pid; w < total_items && ok; w += n_pairs, ++acc_iter) {
        const int a = g.acc_bufs == 2 ? (acc_iter & 1) : 0;
        const uint32_t acc_phase = (uint32_t)(g.acc_bufs == 2 ? (acc_iter >> 1) : acc_iter) & 1u;
        if (!ptx::mbar_wait_hot(&acc_empty_bar[a], acc_phase ^ 1)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(a * acc_cols);
        uint32_t acc = 0;
        for (int kb = 0; kb < kbn; ++kb) {
          if (!ready && !ptx::mbar_wait_hot_addr(full0 + boff, phase)) { ok = false; break; }
          if (dbg && w == pid && (kb == 0 || kb == kbn - 1)) { dbg[kb == 0 ? 2 : 3] = ptx::globaltimer_ns(); dbg[kb == 0 ? 14 : 15] = (unsigned long long)clock64(); }
          const uint32_t cw = w_lo, ca = a_lo, cfree = empty0 + boff;
          w_lo += lo_step; a_lo += lo_step; boff += 8;
          if (boff == bar_end) { boff = 0; phase ^= 1; w_lo = w_lo0; a_lo = a_lo0; }
          // one instruction sequence: test the next stage's barrier, issue this k-block's products, commit them to
          // this stage's "free" barrier (in both blocks), read the test's result
          if (DUAL) ready = ptx::umma_step2_f16_pair(d_tmem, d_tmem + d2_off, cw, cw + up_lo, ca, hi, idesc, acc, cfree, full0 + boff, phase);
          else ready = ptx::umma_step_f16_pair(d_tmem, cw, ca, hi, idesc, acc, cfree, full0 + boff, phase);
          acc = 1;
        }
        if (ok) ptx::umma_commit_pair(&acc_full_bar[a], 3);
      }
      if (!ok) { atomicExch(g.status, -6); abort_flag = 1; }
    }
  } else if (warp >= 2 && warp < 6) {
    // ------------------------------ epilogue (warps 2..5 of both blocks) ------------------------------
    const int quarter = warp & 3;        // TMEM lanes [32 * quarter, 32 * quarter + 32)
    const int fl = quarter * 32 + lane;  // feature within this block's 128
    const int et = threadIdx.x - 64;     // epilogue thread id 0..127
    constexpr bool RESID = EPI == EPI_RESID_NORM;
    constexpr bool SCALED = EPI == EPI_STORE || EPI == EPI_GEGLU;
    ptx::pdl_wait_prior_grids();  // outputs may still be in use by the preceding grid
    const uint32_t acc_empty0 = ptx::mapa_shared(ptx::smem_u32(&acc_empty_bar[0]), 0);
    int acc_iter = 0;
    bool ok = true;
    auto load_old = [&](float (&dst)[CW], int tok, int f) {
      if constexpr (RESID) {
        const float* hp = g.h + (int64_t)tok * g.n_feat + (f < g.n_feat ? f : 0);
#pragma unroll
        for (int j = 0; j < CW; ++j) dst[j] = __ldcg(hp + (int64_t)j * g.n_feat);
      }
    };
    for (int w = pid; w < total_items; w += n_pairs, ++acc_iter) {
      const int ft = (w % n_fpairs) * 2 + rank, tt = w / n_fpairs;
      const int a = g.acc_bufs == 2 ? (acc_iter & 1) : 0;
      const uint32_t acc_phase = (uint32_t)(g.acc_bufs == 2 ? (acc_iter >> 1) : acc_iter) & 1u;
      const int f = ft * TILE_F + fl;
      const int tok0 = tt * g.tile_tok;
      // what does not depend on the accumulator comes before the wait for it: the tokens' 1/rms (from the producer's
      // per-feature-tile sums of squares, added in tile order) and the residual values of the first chunk
      if constexpr (SCALED) {
        epi_bar_sync();  // the previous item's scales have been read
        for (int t = et; t < g.tile_tok; t += 128) {
          float r = 1.f;
          if (g.norm_ssq) {
            const float* sp = g.norm_ssq + tok0 + t;
            float tot = 0.f;
#pragma unroll 4
            for (int i = 0; i < g.norm_tiles; ++i) tot += __ldcg(sp + (int64_t)i * g.ssq_ld);
            r = 1.0f / sqrtf(tot / (float)g.norm_dim + g.eps);
          } else if (g.rowscale) {
            r = g.rowscale[tok0 + t];
          }
          rs_tile[t] = r;
        }
        epi_bar_sync();
      }
      float oldn[CW];
      if constexpr (!RESID) {
#pragma unroll
        for (int j = 0; j < CW; ++j) oldn[j] = 0.f;
      }
      load_old(oldn, tok0, f);
      if (ok) {
        int okw = 1;
        if (lane == 0) okw = ptx::mbar_wait(&acc_full_bar[a], acc_phase) ? 1 : 0;
        okw = __shfl_sync(0xffffffffu, okw, 0);
        if (!okw) ok = false;
      }
      if (ok) {
        for (int spin = 0; spin < 4096 && !ptx::mbar_try_wait(&acc_full_bar[a], acc_phase); ++spin) {}
        ptx::tc_fence_after();
        if (dbg && threadIdx.x == 64 && w == pid) dbg[4] = ptx::globaltimer_ns();
        if (trace && threadIdx.x == 64 && w + n_pairs >= total_items) trace[blockIdx.x * 4 + 3] = ptx::globaltimer_ns();
        const uint32_t t_addr = tmem_base + (uint32_t)(a * acc_cols) + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
        for (int c0 = 0; c0 < g.tile_tok; c0 += CW) {
          float v[CW], v2[CW];
          if constexpr (CW == 32) {
            ptx::tmem_ld_32x32(t_addr + c0, v);
            if (DUAL) ptx::tmem_ld_32x32(t_addr + g.tile_tok + c0, v2);
          } else {
            ptx::tmem_ld_32x16(t_addr + c0, v);
            if (DUAL) ptx::tmem_ld_32x16(t_addr + g.tile_tok + c0, v2);
          }
          ptx::tmem_ld_wait();
          float old[CW];
#pragma unroll
          for (int j = 0; j < CW; ++j) old[j] = oldn[j];
          if (c0 + CW < g.tile_tok) load_old(oldn, tok0 + c0 + CW, f);
          finalize_chunk<DUAL, CW, EPI>(g, v, v2, old, tok0 + c0, f, c0, red, rs_tile + c0);
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (rank == 0) ptx::mbar_arrive(&acc_empty_bar[a]);
          else ptx::mbar_arrive_remote(acc_empty0 + 8u * a);
        }
        if ((EPI == EPI_RESID_NORM || EPI == EPI_EMBED_NORM) && ft < g.n_ftiles)
          finalize_stats(g, min(g.tile_tok, g.n_tok - tok0), tok0, ft, red);
        if (dbg && threadIdx.x == 64 && w == pid) dbg[5] = ptx::globaltimer_ns();
      }
    }
    if (!ok && lane == 0) { atomicExch(g.status, -6); abort_flag = 1; }
  }

  // ------------------------------ teardown ------------------------------
  ptx::tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    // a wait expired: give copies still in flight time to land before the block's memory is released
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) {}
    __syncthreads();
  }
  if (dbg && threadIdx.x == 0) { dbg[6] = ptx::globaltimer_ns(); dbg[13] = (unsigned long long)clock64(); }
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4 + 2] = ptx::globaltimer_ns();
  // neither block leaves (or gives its tensor memory back) while the partner may still read its shared memory or
  // signal its barriers
  ptx::cluster_arrive_release();
  ptx::cluster_wait_acquire();
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, g.tmem_cols);
  }
}

}  // namespace tc
}  // namespace adit
