// Ragged-prefix attention on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// One block handles a tile of 128 query rows of one (request, kv head) group - row r is suffix token
// r / G with query head kvh * G + r % G - against a range of 64-key blocks of the key list
// [prefix 0..P_b) ++ [suffix 0..N).  Per key block:
//   S = Q K^T        tcgen05.mma, M = 128 rows, N = 64 keys, K = head_dim; S lives in TMEM (2 buffers)
//   softmax          8 warps: warps w and w + 4 share the 32 rows of TMEM lane quadrant w and take one half of the
//                    block's 64 columns each, so that every scheduler has two warps to hide the per-block latencies
//                    (barrier tests, tcgen05.ld) of the other; a thread's 32 scores come out of TMEM with
//                    tcgen05.ld, row max and row sum are plain per-thread loops, the two half-row maxima are
//                    exchanged through shared memory (bounded mbarrier hand-shake) and both threads then take the
//                    same decisions; exp2 with log2(e)/sqrt(dh) folded into the scale; P goes back to TENSOR
//                    memory as bf16 pairs (tcgen05.st): no shared-memory round trip, no proxy fence
//   O += P V         tcgen05.mma with the A operand (P) in tensor memory, M = 128, N = head_dim, K = 64 keys; V is
//                    used as stored ([key][channel], an MN-major operand), O accumulates in TMEM
// O is only rescaled when a row's running maximum grows by more than 2^8 (the reference maximum is kept
// otherwise), which keeps the TMEM read-modify-write off the common path.
//
// The key list of a request is [prefix 0..P_b), padded with masked keys to a multiple of 64, then the suffix keys:
// every 64-key block is then either a box of the request's prefix cache or a box of this step's suffix K/V rows, and
// both come in by TMA (cp.async.bulk.tensor, 128-byte swizzle = the layout the MMA descriptors expect), issued by
// one thread per operand.  The prefix cache is described by a per-request tensor map whose row extent is the prefix
// length: rows at or beyond it are never read (the copy engine writes zeros), and their scores are masked to -inf.
// The K ring (two stages) and the V ring (three: V is needed last in a block's chain, and its ring has to cover the
// copies' latency of about a microsecond) are released separately - a K stage as soon as its Q K^T has completed, a V
// stage after its P V - and P is double-buffered, so the softmax of block n only depends on the tensor core through
// S(n), P V(n - 2) and, when a row maximum forces a rescale of O, P V(n - 1).  Tensor memory: O 256 columns, S 2 x 64,
// P 3 x 32.  Shared memory at head_dim 256: Q 64 KB + 5 stages of 32 KB + 3 KB of barriers = the 227 KB of a block.
// Every mbarrier wait is bounded.  With more than one key split the block writes its unnormalised
// partial (O as bf16, m, l) and the merge kernel combines the splits in fixed order.
#pragma once
#include "attention.cuh"
#include "common.cuh"
#include "ptx.cuh"

namespace adit {
namespace attn {

constexpr int TC_ROWS = 128;
// warps 0-7 softmax (warps w and w + 4 share 32 query rows and take one half of a key block's columns each), 8 issuer of
// Q K^T (+ TMEM owner), 9 issuer of P V, 10 K copies, 11 V copies
constexpr int TC_THREADS = 384;
constexpr int P_BUFS = 3;    // probability buffers in tensor memory: block n may be written while P V(n - 1), P V(n - 2) are pending
constexpr int V_STAGES = 3;  // V is consumed last in a key block's chain: its ring has to cover the copies' latency

template <int DH>
constexpr size_t attn_tc_smem_bytes() {
  // Q tile + two K stages + three V stages (the probabilities live in tensor memory).  The dynamic array is declared
  // 1024-byte aligned, so it starts at the first such offset behind the kernel's static shared memory (at most 3 KB:
  // with head_dim 256 the sum is exactly the 227 KB a block may have); smaller head dimensions keep a kilobyte of
  // slack for a run-time round-up.
  return (size_t)TC_ROWS * DH * 2 + (2 + V_STAGES) * (size_t)KEY_BLOCK * DH * 2 + (DH >= 256 ? 0 : 1024);
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 16-byte chunk c of row r of a [rows][64]-element (128-byte rows) swizzled box
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// INSTR: phase stamps and launch trace compiled in (test and measurement aids; the plain instantiation is smaller
// and starts faster).
// PARTIAL: the key list of a row tile is split over several blocks (a.splits > 1): unnormalised partial outputs.
// QTMA: the query tile comes in by TMA (the usual case); otherwise by per-thread copies.
template <int DH, bool INSTR = false, bool PARTIAL = false, bool QTMA = true>
__global__ void __launch_bounds__(TC_THREADS, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                const __grid_constant__ CUtensorMap map_sfx, AttnArgs a,
                                                                const PrefixTable* __restrict__ ptp) {
  constexpr int KV_BYTES = KEY_BLOCK * DH * 2;
  constexpr int Q_BYTES = TC_ROWS * DH * 2;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t k_full[2], v_full[V_STAGES], k_empty[2], v_empty[V_STAGES], s_full[2], s_empty[2], p_full[P_BUFS], pv_done[P_BUFS], q_full, o_done;
  __shared__ __align__(8) uint64_t pair_bar[4];  // hand-shake of the two softmax warps that share 32 rows
  __shared__ float xch_max[2][2][TC_ROWS];       // [block parity][column half][row]: half-row maxima (and, after the
                                                 // last block, the half-row sums in the buffer of the other parity)
  __shared__ uint32_t tmem_base_smem;
  __shared__ volatile int abort_flag;

  ptx::pdl_launch_dependents();
  unsigned long long* const trace = INSTR ? a.trace : nullptr;
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4] = ptx::globaltimer_ns();
  unsigned long long* const dbg = (INSTR && a.dbg) ? a.dbg + (size_t)blockIdx.x * 16 : nullptr;
  if (dbg && threadIdx.x == 0) dbg[0] = ptx::globaltimer_ns();
  unsigned long long* const dlog = (INSTR && a.dbg && blockIdx.x == 0) ? a.dbg + 8192 : nullptr;  // per-key-block log of block 0
  uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  if (DH >= 256 && base != smem_raw) {  // (no slack at this size: never expected, and nothing has been touched yet)
    if (threadIdx.x == 0 && a.status) atomicExch(a.status, -5);
    return;
  }
  uint8_t* sQ = base;                       // DH / 64 boxes [128 rows][64 ch]
  uint8_t* sK = sQ + Q_BYTES;               // 2 stages x DH / 64 boxes [64 keys][64 ch]
  uint8_t* sV = sK + 2 * KV_BYTES;          // V_STAGES stages, same boxes
  uint8_t* stage = sK;                      // output staging, aliases sK, sV once the products are done
  constexpr int STAGE_STRIDE = DH * 2 + 16; // bf16 row + 16 bytes against bank conflicts
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const PrefixTable& pt = *ptp;
  const int G = a.n_q_heads / a.n_kv_heads;
  const int R = a.n_tokens * G;
  const int k_off = a.n_q_heads * DH, v_off = k_off + a.n_kv_heads * DH;
  const int n_splits = PARTIAL ? a.splits : 1;
  const int n_items = a.batch * a.n_kv_heads * a.n_row_tiles * n_splits;

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&k_full[s], 1);  // the loading thread's expect-tx arrival; the copies count the bytes
      ptx::mbar_init(&k_empty[s], 1);
      ptx::mbar_init(&s_full[s], 1);
      ptx::mbar_init(&s_empty[s], 8);  // one arrival per softmax warp (separate arrivals of every thread on one barrier word are slow)
    }
    for (int v = 0; v < V_STAGES; ++v) { ptx::mbar_init(&v_full[v], 1); ptx::mbar_init(&v_empty[v], 1); }
    for (int v = 0; v < P_BUFS; ++v) { ptx::mbar_init(&p_full[v], 8); ptx::mbar_init(&pv_done[v], 1); }
    for (int w = 0; w < 4; ++w) ptx::mbar_init(&pair_bar[w], 2);
    ptx::mbar_init(&q_full, 1);
    ptx::mbar_init(&o_done, 1);  // all P V products of a work item complete (once per item: no parity doubt for early waiters)
    if (QTMA) ptx::prefetch_tensormap(&map_q);
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 8) {
    ptx::tmem_alloc(&tmem_base_smem, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = tmem_base_smem;
  const uint32_t tm_o = tmem;             // O: DH columns
  const uint32_t tm_s = tmem + 256;       // S: 2 x 64 columns
  const uint32_t tm_p = tmem + 384;       // P: P_BUFS x 32 columns (bf16 pairs: the A operand of P V, read straight from here)
  // The prefix caches do not depend on the preceding kernel (only Q and the suffix K/V do): the loader
  // warps start on key blocks that lie wholly in the prefix right away and wait for the preceding grid only
  // when they first need a suffix row; every other warp waits once it has worked out its first work item.
  const bool is_loader = (threadIdx.x >> 5) >= 10;
  bool waited = false;

  // Barrier phases run on across work items: these counters are kept per role.
  uint32_t kv_cnt = 0;   // key blocks processed so far by this role (block n uses stage, S, P buffer and barriers n & 1)
  uint32_t q_cnt = 0;    // query tiles loaded so far
  uint32_t pair_cnt = 0; // hand-shakes of this softmax warp with its partner so far
  bool ok = true;

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    int t = item;
    const int split = PARTIAL ? t % n_splits : 0;
    if (PARTIAL) t /= n_splits;
    const int rt = t % a.n_row_tiles; t /= a.n_row_tiles;
    const int kvh = t % a.n_kv_heads;
    const int b = t / a.n_kv_heads;
    const int plen = pt.len[b];
    const int npb = (plen + KEY_BLOCK - 1) / KEY_BLOCK;                       // prefix blocks (the last one padded)
    const int nkb = npb + (a.n_tokens + KEY_BLOCK - 1) / KEY_BLOCK;           // + suffix blocks
    const int kb0 = PARTIAL ? (int)((int64_t)split * nkb / n_splits) : 0;
    const int kb1 = PARTIAL ? (int)((int64_t)(split + 1) * nkb / n_splits) : nkb;
    const int nb = kb1 - kb0;
    const int64_t tok0 = (int64_t)b * a.n_tokens;

    // ---- Q tile (all threads), visible to the tensor core before the first product ----
    if (!waited && !is_loader) {
      ptx::pdl_wait_prior_grids();
      waited = true;
      if (trace && threadIdx.x == 0) trace[blockIdx.x * 4 + 1] = ptx::globaltimer_ns();
      if (dbg && threadIdx.x == 0) dbg[1] = ptx::globaltimer_ns();
    }
    // previous item completely finished (its last PV has been waited for by the softmax warps); leave together on abort
    if (item != (int)blockIdx.x && __syncthreads_or(abort_flag)) break;
    if constexpr (QTMA) {
      // rows of the tile are (token, head-in-group) pairs in token-major order: one box per 64 channels
      if (tid == 0 && nb > 0) {
        ptx::mbar_arrive_expect_tx(&q_full, Q_BYTES);
        for (int j = 0; j < DH / 64; ++j)
          ptx::tma_load_3d(sQ + j * (TC_ROWS * 128), &map_q, j * 64, kvh * G, (int)tok0 + rt * (TC_ROWS / G), &q_full);
      }
    } else {
      if (!waited) { ptx::pdl_wait_prior_grids(); waited = true; }
      for (int e = tid; e < TC_ROWS * (DH / 8); e += TC_THREADS) {
        const int r = e / (DH / 8), c = e % (DH / 8);
        const int gr = rt * TC_ROWS + r;
        uint8_t* dst = sQ + (c >> 3) * (TC_ROWS * 128) + swz(r, c & 7);
        if (gr < R) {
          const int tok = gr / G, hq = kvh * G + gr % G;
          cp_async16(dst, a.qkv + (tok0 + tok) * a.ldqkv + hq * DH + c * 8);
        } else {
          *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
        }
      }
      cp_async_commit();
      cp_async_wait_all();
      ptx::fence_proxy_async();
      __syncthreads();
    }
    if (dbg && threadIdx.x == 0 && item == (int)blockIdx.x) dbg[2] = ptx::globaltimer_ns();

    if (warp >= 10) {
      // ------------------------------ K copies (warp 10) and V copies (warp 11) ------------------------------
      const int which = warp == 11 ? 1 : 0;
      uint64_t* empty_bar = which ? v_empty : k_empty;
      uint64_t* full_bar = which ? v_full : k_full;
      uint8_t* ring = which ? sV : sK;
      if (lane == 0) {
        // one thread per operand issues the copies: dh / 64 boxes of 64 keys x 64 channels per block
        const int plane = (a.layer * 2 + which) * a.n_kv_heads + kvh;
        const CUtensorMap* pm = a.kv_maps + b;
        if (npb > 0 && kb0 < npb) ptx::tensormap_acquire(pm);
        for (int i = 0; i < nb && ok; ++i) {
          const uint32_t n = kv_cnt + i;
          const int s = which ? (int)(n % V_STAGES) : (int)(n & 1);
          const uint32_t par = which ? ((n / V_STAGES) & 1) : ((n >> 1) & 1);
          if (!ptx::mbar_wait(&empty_bar[s], par ^ 1)) { ok = false; break; }
          uint8_t* dst = ring + s * KV_BYTES;
          const int blk = kb0 + i;
          ptx::mbar_arrive_expect_tx(&full_bar[s], KV_BYTES);
          if (blk < npb) {
#pragma unroll
            for (int j = 0; j < DH / 64; ++j)
              ptx::tma_load_3d(dst + j * (KEY_BLOCK * 128), pm, j * 64, blk * KEY_BLOCK, plane, &full_bar[s]);
          } else {
            if (!waited) { ptx::pdl_wait_prior_grids(); waited = true; }  // only the suffix rows depend on the preceding grid
            const int rowg = (int)tok0 + (blk - npb) * KEY_BLOCK;
#pragma unroll
            for (int j = 0; j < DH / 64; ++j)
              ptx::tma_load_2d(dst + j * (KEY_BLOCK * 128), &map_sfx, (which ? v_off : k_off) + kvh * DH + j * 64, rowg, &full_bar[s]);
          }
          if (dbg && which == 0 && item == (int)blockIdx.x && i < 2) dbg[3 + i] = ptx::globaltimer_ns();
          if (dlog && which == 0 && item == 0 && i < 32) dlog[i * 4 + 0] = ptx::globaltimer_ns();
        }
        if (!ok) { if (a.status) atomicExch(a.status, -6); abort_flag = 1; }
      }
      kv_cnt += nb;
    } else if (warp == 8) {
      // ------------------------------ issuer of S = Q K^T ------------------------------
      // Issuing a product costs its thread about 80 cycles; a key block needs head_dim / 16 of them for the
      // scores and 4 for P V, so the two kinds have a thread each.  Scores run ahead of the softmax as far as
      // the K stages and the two S buffers allow.
      if (lane == 0) {
        const uint32_t idesc_s = ptx::idesc_bf16_f32(TC_ROWS, KEY_BLOCK);
        const uint32_t desc_hi = ptx::smem_desc_hi_sw128();
        const uint32_t q_lo0 = ptx::smem_desc_lo(ptx::smem_u32(sQ)), k_lo0 = ptx::smem_desc_lo(ptx::smem_u32(sK));
        if (nb > 0 && QTMA && !ptx::mbar_wait(&q_full, q_cnt & 1)) ok = false;
        for (int i = 0; i < nb && ok; ++i) {
          const uint32_t n = kv_cnt + i;
          const int s = n & 1;
          if (!ptx::mbar_wait(&k_full[s], (n >> 1) & 1) || !ptx::mbar_wait(&s_empty[s], ((n >> 1) & 1) ^ 1)) { ok = false; break; }
          ptx::tc_fence_after();
          // head_dim / 64 groups of four products: descriptor halves in registers, one instruction sequence per group
          // (this thread's own instruction latencies are what a key block's scores cost)
          const uint32_t k_lo = k_lo0 + (uint32_t)s * (KV_BYTES >> 4);
#pragma unroll
          for (int j = 0; j < DH / 64; ++j)
            ptx::umma_kblock_f16(tm_s + s * KEY_BLOCK, q_lo0 + j * (TC_ROWS * 128 >> 4), k_lo + j * (KEY_BLOCK * 128 >> 4), desc_hi, idesc_s,
                                 j > 0 ? 1u : 0u);
          ptx::umma_commit(&s_full[s]);
          ptx::umma_commit(&k_empty[s]);  // the K stage is free as soon as these products have read it
        }
        if (!ok) { if (a.status) atomicExch(a.status, -6); abort_flag = 1; }
      }
      kv_cnt += nb;
    } else if (warp == 9) {
      // ------------------------------ issuer of O += P V ------------------------------
      if (lane == 0) {
        const uint32_t idesc_o = ptx::idesc_bf16_f32(TC_ROWS, DH) | (1u << 16);  // B (= V) is MN-major
        for (int i = 0; i < nb && ok; ++i) {
          const uint32_t n = kv_cnt + i;
          const int vs = (int)(n % V_STAGES);
          const int ps = (int)(n % P_BUFS);
          if (!ptx::mbar_wait(&v_full[vs], (n / V_STAGES) & 1) || !ptx::mbar_wait_hot(&p_full[ps], (n / P_BUFS) & 1)) { ok = false; break; }
          ptx::tc_fence_after();
          // P is read out of tensor memory (8 columns of bf16 pairs per product), V out of its stage
          const uint32_t pa = tm_p + ps * (KEY_BLOCK / 2), va = ptx::smem_u32(sV + vs * KV_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < KEY_BLOCK / 16; ++k4)
            ptx::umma_f16_ta(tm_o, pa + k4 * 8, ptx::smem_desc_mn_sw128(va + k4 * 16 * 128, KEY_BLOCK * 128), idesc_o,
                             (i > 0 || k4 > 0) ? 1u : 0u);
          ptx::umma_commit(&pv_done[ps]);
          ptx::umma_commit(&v_empty[vs]);
          if (i == nb - 1) ptx::umma_commit(&o_done);
          if (dlog && item == 0 && i < 32) dlog[i * 4 + 3] = ptx::globaltimer_ns();
        }
        if (!ok) { if (a.status) atomicExch(a.status, -6); abort_flag = 1; }
      }
      kv_cnt += nb;
    } else {
      // ------------------------------ softmax / output (warps 0-7) ------------------------------
      // Thread = (query row, column half): warps w and w + 4 can both read the TMEM lanes of rows 32 w .. 32 w + 31 and
      // take columns [0, 32) and [32, 64) of every key block (and the lower / upper half of the output channels).  With
      // one warp per scheduler the per-block latencies (barrier tests, tensor-memory loads) lay bare; two warps hide them
      // for each other.  The row maximum is the only thing the halves have to agree on: they exchange their half-row
      // maxima through shared memory once per block and then take identical decisions.
      const int half = warp >> 2, wq = warp & 3;
      const int row = wq * 32 + lane;  // 0..127, also the TMEM lane
      const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
      constexpr int HB = KEY_BLOCK / 2;  // columns of a key block per thread
      // Wait of a whole warp: one non-blocking test by every lane when the phase is already complete (a barrier
      // instruction costs over a hundred cycles), otherwise lane 0 waits with the time limit and the others follow.
      auto warp_wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        if (__all_sync(0xffffffffu, ptx::mbar_test_wait(bar, parity))) return true;
        int okw = 1;
        if (lane == 0) okw = ptx::mbar_wait(bar, parity) ? 1 : 0;
        okw = __shfl_sync(0xffffffffu, okw, 0);
        if (!okw) return false;
        for (int spin = 0; spin < 4096 && !ptx::mbar_try_wait(bar, parity); ++spin) {}
        return true;
      };
      // Bounded hand-shake with the warp that shares this warp's rows (an mbarrier, not bar.sync: a warp that gave up
      // on a wait must not strand its partner).  Orders this warp's shared-memory writes before the partner's reads.
      auto pair_sync = [&]() -> bool {
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&pair_bar[wq]);
        const bool okp = warp_wait(&pair_bar[wq], pair_cnt & 1);
        ++pair_cnt;
        return okp;
      };
      float m_ref = -INFINITY, l = 0.f;
      for (int i = 0; i < nb && ok; ++i) {
        const uint32_t n = kv_cnt + i;
        const int s = n & 1;
        if (!warp_wait(&s_full[s], (n >> 1) & 1)) { ok = false; break; }
        ptx::tc_fence_after();
        if (dbg && tid == 0 && item == (int)blockIdx.x && i < 2) dbg[5 + 2 * i] = ptx::globaltimer_ns();
        if (dlog && tid == 0 && item == 0 && i < 32) dlog[i * 4 + 1] = ptx::globaltimer_ns();
        float sc[HB];
        ptx::tmem_ld_32x32(tm_s + s * KEY_BLOCK + half * HB + lane_addr, sc);
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&s_empty[s]);
        // block maximum of the raw scores (the scale is positive, so it commutes with max); only the last
        // block of a key list can hold columns outside it, which are masked to -inf
        // keys of this block that exist: a prefix block ends at prefix_len, a suffix block at the token count
        const int blk = kb0 + i;
        const int nvalid = blk < npb ? min(KEY_BLOCK, plen - blk * KEY_BLOCK) : min(KEY_BLOCK, a.n_tokens - (blk - npb) * KEY_BLOCK);
        if (nvalid < KEY_BLOCK) {
#pragma unroll
          for (int j = 0; j < HB; ++j)
            if (half * HB + j >= nvalid) sc[j] = -INFINITY;
        }
        // variant: the state token's rows (token 0 of the request: rows 0 .. G-1 of row tile 0) see, of the suffix,
        // the state token's own key only
        if (a.state_mask && rt * TC_ROWS + row < G && blk >= npb) {
          const int first = (blk - npb) * KEY_BLOCK + half * HB;
#pragma unroll
          for (int j = 0; j < HB; ++j)
            if (first + j > 0) sc[j] = -INFINITY;
        }
        // (four independent chains: a thread cannot hide the latency of one long chain)
        float mx[4] = {sc[0], sc[1], sc[2], sc[3]};
#pragma unroll
        for (int j = 4; j < HB; j += 4) {
          mx[0] = fmaxf(mx[0], sc[j]); mx[1] = fmaxf(mx[1], sc[j + 1]);
          mx[2] = fmaxf(mx[2], sc[j + 2]); mx[3] = fmaxf(mx[3], sc[j + 3]);
        }
        const float mhalf = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        xch_max[i & 1][half][row] = mhalf;
        if (!pair_sync()) { ok = false; break; }
        const float mraw = fmaxf(mhalf, xch_max[i & 1][half ^ 1][row]);
        const float mb = mraw * a.scale_log2;
        // the reference maximum only moves when it would otherwise be exceeded by more than 2^8
        float corr = 1.f;
        const bool grow = mb > m_ref + 8.f;
        if (grow) {
          corr = exp2f(m_ref - mb);  // 0 on the first block (m_ref = -inf)
          m_ref = mb;
          l *= corr;
        }
        // O may only be rescaled once the previous P V has completed (rare after the first blocks); each half
        // rescales its half of the channels (both warps of a pair see the same rows, hence the same decision)
        if (i > 0 && __any_sync(0xffffffffu, grow)) {
          const uint32_t q = n - 1;
          if (!warp_wait(&pv_done[q % P_BUFS], (q / P_BUFS) & 1)) { ok = false; break; }
          ptx::tc_fence_after();
#pragma unroll 1
          for (int c0 = half * (DH / 2); c0 < (half + 1) * (DH / 2); c0 += 32) {
            float o[32];
            ptx::tmem_ld_32x32(tm_o + c0 + lane_addr, o);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] *= corr;
            ptx::tmem_st_32x32(tm_o + c0 + lane_addr, o);
          }
          ptx::tmem_st_wait();
          ptx::tc_fence_before();
        }
        // this block's P buffer was last read by the P V three blocks back
        if (i >= P_BUFS) {
          const uint32_t q = n - P_BUFS;
          if (!warp_wait(&pv_done[q % P_BUFS], (q / P_BUFS) & 1)) { ok = false; break; }
        }
        // (a key range whose keys are all masked for this row leaves the reference maximum at -inf: subtract 0 then,
        // so that the probabilities are exp2(-inf) = 0 and not NaN)
        const float m_sub = m_ref == -INFINITY ? 0.f : m_ref;
        // probabilities -> bf16 pairs -> tensor memory: this thread's 32 keys are 16 columns of its row (lane)
        float rs[4] = {0.f, 0.f, 0.f, 0.f};  // partial row sums, added up in a fixed order
        uint32_t pw[HB / 2];
#pragma unroll
        for (int c = 0; c < HB / 8; ++c) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float p0 = ex2(fmaf(sc[c * 8 + 2 * q], a.scale_log2, -m_sub)), p1 = ex2(fmaf(sc[c * 8 + 2 * q + 1], a.scale_log2, -m_sub));
            rs[q] += p0 + p1;
            pw[c * 4 + q] = pack_bf16(p0, p1);
          }
        }
        l += (rs[0] + rs[1]) + (rs[2] + rs[3]);
        const int ps = (int)(n % P_BUFS);
        ptx::tmem_st_32x16(tm_p + ps * (KEY_BLOCK / 2) + half * (HB / 2) + lane_addr, pw);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&p_full[ps]);
        if (dbg && tid == 0 && item == (int)blockIdx.x && i < 2) dbg[6 + 2 * i] = ptx::globaltimer_ns();
        if (dlog && tid == 0 && item == 0 && i < 32) dlog[i * 4 + 2] = ptx::globaltimer_ns();
      }
      // the row sum: this half's part plus the partner's, lower half first
      if (ok && nb > 0) {
        // (the buffer of parity nb & 1 was last read one hand-shake ago)
        xch_max[nb & 1][half][row] = l;
        if (!pair_sync()) ok = false;
        l = xch_max[nb & 1][0][row] + xch_max[nb & 1][1][row];
      }
      // ---- output ----
      if (ok && nb > 0) {
        const uint32_t q = kv_cnt + nb - 1;
        if (!warp_wait(&pv_done[q % P_BUFS], (q / P_BUFS) & 1)) ok = false;
        ptx::tc_fence_after();
      }
      if (dbg && tid == 0 && item == (int)blockIdx.x) dbg[9] = ptx::globaltimer_ns();
      // Each thread owns half a row, so direct stores would touch 32 different lines per instruction: the
      // rows are staged in shared memory (the K/V/P buffers are free now) and written out by the whole block
      // with contiguous 16-byte stores.
      const int gr = rt * TC_ROWS + row;
      const bool row_ok = gr < R;
      const float inv = PARTIAL ? 1.0f : 1.0f / l;
      uint8_t* srow = stage + (size_t)row * STAGE_STRIDE;
#pragma unroll 1
      for (int c0 = half * (DH / 2); c0 < (half + 1) * (DH / 2); c0 += 32) {
        float o[32];
        if (nb > 0 && ok) {
          ptx::tmem_ld_32x32(tm_o + c0 + lane_addr, o);
          ptx::tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = 0.f;
        }
        // final rows are normalised; partial rows of a key split stay relative to the row's reference maximum
#pragma unroll
        for (int j = 0; j < 32; j += 8)
          *reinterpret_cast<uint4*>(srow + (c0 + j) * 2) =
              make_uint4(pack_bf16(o[j] * inv, o[j + 1] * inv), pack_bf16(o[j + 2] * inv, o[j + 3] * inv),
                         pack_bf16(o[j + 4] * inv, o[j + 5] * inv), pack_bf16(o[j + 6] * inv, o[j + 7] * inv));
      }
      if (PARTIAL && row_ok && half == 0) {
        const int tok = gr / G, hq = kvh * G + gr % G;
        const int64_t qrow = (tok0 + tok) * a.n_q_heads + hq;
        const int64_t n_qrows = (int64_t)a.batch * a.n_tokens * a.n_q_heads;
        float* ml = a.part_ml + ((int64_t)split * n_qrows + qrow) * 2;
        ml[0] = m_ref;
        ml[1] = l;
      }
      if (dbg && tid == 0 && item == (int)blockIdx.x) dbg[10] = ptx::globaltimer_ns();
      ptx::tc_fence_before();
      kv_cnt += nb;
      if (!ok && lane == 0) { if (a.status) atomicExch(a.status, -6); abort_flag = 1; }
    }
    if (nb > 0) ++q_cnt;
    // ---- staged rows -> global memory: one warp per row, one 16-byte piece per lane and pass ----
    __syncthreads();
    if (dbg && tid == 0 && item == (int)blockIdx.x) dbg[12] = ptx::globaltimer_ns();
    if (trace && tid == 0) trace[blockIdx.x * 4 + 3] = ptx::globaltimer_ns();
    {
      const int rows_valid = min(TC_ROWS, R - rt * TC_ROWS);
      const int64_t n_qrows = (int64_t)a.batch * a.n_tokens * a.n_q_heads;
      const int g_shift = (G & (G - 1)) == 0 ? __ffs(G) - 1 : -1;  // group size is a power of two in practice
      for (int r = warp; r < rows_valid; r += TC_THREADS / 32) {
        const int gr = rt * TC_ROWS + r;
        const int tok = g_shift >= 0 ? (gr >> g_shift) : gr / G;
        const int hq = kvh * G + (gr - tok * G);
        const uint8_t* src = stage + (size_t)r * STAGE_STRIDE;
        uint8_t* dst = !PARTIAL
                           ? reinterpret_cast<uint8_t*>(a.att + (tok0 + tok) * a.ldatt + hq * DH)
                           : reinterpret_cast<uint8_t*>((bf16*)a.part_o + ((int64_t)split * n_qrows + (tok0 + tok) * a.n_q_heads + hq) * DH);
#pragma unroll
        for (int c = 0; c < DH * 2 / 16; c += 32)
          if (c + lane < DH * 2 / 16)
            *reinterpret_cast<uint4*>(dst + (c + lane) * 16) = *reinterpret_cast<const uint4*>(src + (c + lane) * 16);
      }
    }
    if (dbg && tid == 0 && item == (int)blockIdx.x) dbg[13] = ptx::globaltimer_ns();
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) {}
    __syncthreads();
  }
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4 + 2] = ptx::globaltimer_ns();
  if (dbg && threadIdx.x == 0) dbg[11] = ptx::globaltimer_ns();
  if (warp == 8) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, 512);
  }
}

}  // namespace attn
}  // namespace adit
