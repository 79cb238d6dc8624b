// Persistent bf16 projection kernel on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
// Orientation ("swap-AB"): the weight matrix W[n_feat, K] (K contiguous) is the MMA's M-side operand
// in tiles of 128 output features; the activations A[n_tok, K] (K contiguous) are the N-side operand
// in tiles of `tile_tok` tokens (any multiple of 16 up to 256).  The accumulator D[feature, token]
// lives in tensor memory: lane = feature, column = token, so a batch-1 call (51 tokens) still uses
// full 128-row MMAs and the weight stream is the only large operand.
//
// k-split across a thread-block cluster: when there are fewer output tiles than SMs, `splits` blocks
// of one cluster share an output tile, each multiplying its own slice of K.  The partial
// accumulators are exchanged through distributed shared memory (every block owns tile_tok / splits
// tokens and receives the other blocks' values for them), summed in rank order - the result is
// bitwise reproducible and independent of the grid size - and only then does the epilogue run, so
// no partial sums go through global memory and no separate reduction kernel is needed.
//
// Epilogues: bf16 store with per-token scale (RMSNorm folded: gain in the weights, 1/rms here),
// SiLU with an added vector, GeGLU on a gate/up pair of accumulators, fp32 store, and two residual
// forms that write the fp32 residual stream, its bf16 copy (the next projection's operand) and the
// per-token sums of squares per feature tile, from which the next projection's epilogue derives 1/rms.
//
// Warp roles (256 threads): warps 0 and 6 = TMA producers (weight tiles, activation tiles), warp 1 = TMEM
// allocator + MMA issuer, warp 7 = second MMA issuer, warps 2..5 = epilogue (each owns the 32 TMEM lanes of its
// warp-id modulo 4).  Issuing a product costs its thread about 80 cycles whatever the tile width, so narrow
// tiles are issue-bound: with two issuers the k-blocks alternate between them, each adding into
// accumulators of its own, which the epilogue sums.  Shared-memory stages
// and the two TMEM accumulator buffers are handed over with mbarriers; every mbarrier wait is bounded.
#pragma once
#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"

namespace adit {
namespace tc {

constexpr int TILE_F = 128;    // output features per tile (MMA M)
constexpr int TILE_K = 64;     // k elements per pipeline stage: 128 bytes of bf16, one swizzle row
constexpr int UMMA_K = 16;     // k elements per tcgen05.mma
constexpr int MAX_STAGES = 12;
constexpr int GEMM_THREADS = 256;
constexpr int SMEM_BUDGET = 216 * 1024;  // dynamic shared memory: stage ring + cluster exchange buffer

enum : int { EPI_RESID_NORM = 6, EPI_EMBED_NORM = 7, EPI_STORE_PLANES = 8 };

struct GemmArgs {
  int n_feat;    // output features (DUAL: per matrix; the packed matrix has 2 * n_feat rows)
  int n_tok;     // valid token rows of A
  int kb_total;  // K / 64
  int tile_tok;  // tokens per tile (multiple of 16, <= 256; a multiple of 8 * splits)
  int n_ftiles, n_ttiles;
  int splits;    // k-split = cluster size (1, 2, 4 or 8)
  int stages;
  int acc_bufs;        // accumulator buffers in tensor memory: 2, or 1 when a tile needs more than half of it
  int issuers;         // MMA-issuing threads: 1 or 2
  uint32_t tmem_cols;  // power of two >= acc_bufs accumulator buffers
  uint32_t ring_bytes; // stages * stage bytes; the exchange buffer follows
  int epi;
  void* out;             // EPI_STORE / SILU / GEGLU: bf16 [n_tok, ldo]; EPI_STORE_F32: fp32
  int ldo;
  const float* rowscale; // [n_tok] or null (EPI_STORE only; ignored when norm_ssq is set)
  const float* norm_ssq; // EPI_STORE / EPI_GEGLU: [norm_tiles][ssq_ld] sums of squares of the operand rows; the epilogue
  int norm_tiles;        //   multiplies token t by 1/sqrt(sum_i norm_ssq[i][t] / norm_dim + eps) (RMSNorm with folded gain)
  int norm_dim;
  const float* bias;     // [n_feat] or null
  // residual epilogues (n_feat == width of the residual stream)
  float* h;              // fp32 residual stream [rows, n_feat]
  bf16* hb;              // its bf16 copy
  float* ssq;            // [n_ftiles][ssq_ld] per-tile sums of squares of the new rows
  int ssq_ld;
  float eps;
  int horizon;           // EPI_EMBED_NORM: action row m -> token row m + m / horizon + 1
  int plane_w;           // EPI_STORE_PLANES: feature f of token t goes to out[(f / plane_w) * plane_stride + t * plane_w + f % plane_w]
  int64_t plane_stride;  //   (bf16; a K/V cache laid out as planes of [rows][plane_w]); tokens >= n_tok are not stored
  int* status;           // device-visible status word (ADIT_E_TIMEOUT = -6 on an expired wait)
  int debug_withhold;    // test aid (WITHHOLD instantiation only): when n > 0, block 0's token copy of its n-th k-block is never issued
  unsigned long long* dbg;  // optional [grid][16] globaltimer stamps (test aid)
  unsigned long long* trace;  // optional [grid][4]: block start, predecessor-wait released, end, last accumulator complete (%globaltimer ns)
};

__device__ __forceinline__ float gelu_tanh_fast(float y) {
  const float c = 0.7978845608028654f;
  float t;
  float a = c * (y + 0.044715f * y * y * y);
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(a));
  return 0.5f * y * (1.0f + t);
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Sum over the 32 lanes of a warp of NT values per lane (NT = 8, 16 or 32), in the order of an xor-butterfly
// (offsets 16, 8, 4, 2, 1), but keeping only half of the values at every step: NT - 1 + log2(32 / NT) shuffles
// instead of 5 NT.  On return lane l holds in sq[0] the total of value index l / (32 / NT).
template <int NT>
__device__ __forceinline__ void warp_sum_transposed(float (&sq)[NT], int lane) {
  int n = NT;
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    if (n > 1) {
      const bool upper = (lane & off) != 0;
      n >>= 1;
#pragma unroll
      for (int j = 0; j < NT / 2; ++j) {
        if (j < n) {
          const float send = upper ? sq[j] : sq[j + n];
          const float keep = upper ? sq[j + n] : sq[j];
          sq[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
      }
    } else {
      sq[0] += __shfl_xor_sync(0xffffffffu, sq[0], off);
    }
  }
}

// Final values of one thread (feature f) for NT consecutive tokens starting at tok_base.
// Straight-line, predicate-free code: one address computation and one store per token.  Tokens at or
// beyond n_tok are stored too - every output buffer has padding rows for them - because a guard per
// token turns into a chain of slow branches in the single epilogue warp of each scheduler.
// `old` holds the residual stream's current values for these tokens (EPI_RESID_NORM; fetched by the caller
// ahead of time so that the load latency is not paid here), `rs` the per-token scales in shared memory.
template <bool DUAL, int NT, int EPI>
__device__ __forceinline__ void finalize_chunk(const GemmArgs& g, const float (&v)[NT], const float (&v2)[NT],
                                               const float (&old)[NT], int tok_base, int f, int range_off,
                                               float* red /*[4][256]*/, const float* rs /*[NT], shared*/) {
  const bool f_ok = f < g.n_feat;
  if constexpr (EPI == EPI_RESID_NORM || EPI == EPI_EMBED_NORM) {
    // ---- residual stream update + statistics for the next RMSNorm (all 128 epilogue threads take part) ----
    const int lane = threadIdx.x & 31, ew = (threadIdx.x >> 5) & 3;
    constexpr bool embed = EPI == EPI_EMBED_NORM;
    const int64_t ld = g.n_feat;
    float sq[NT];
    if (f_ok) {
      if (embed) {
        const float b = g.bias[f];
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const int tok = tok_base + j;
          const int64_t row = tok + tok / g.horizon + 1;
          const float hv = v[j] + b;
          g.h[row * ld + f] = hv;
          g.hb[row * ld + f] = __float2bfloat16_rn(hv);
          sq[j] = hv * hv;
        }
      } else {
        float* hp = g.h + (int64_t)tok_base * ld + f;
        bf16* bp = g.hb + (int64_t)tok_base * ld + f;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const float hv = old[j] + v[j];
          hp[j * ld] = hv;
          bp[j * ld] = __float2bfloat16_rn(hv);
          sq[j] = hv * hv;
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < NT; ++j) sq[j] = 0.f;
    }
    // sum of squares over this warp's 32 features (fixed tree); the four warps and the feature
    // tiles are combined once per token range by finalize_stats
    warp_sum_transposed<NT>(sq, lane);
    constexpr int LPT = 32 / NT;  // lanes per token
    if ((lane & (LPT - 1)) == 0) red[ew * 256 + range_off + lane / LPT] = sq[0];
  }
  if constexpr (EPI != EPI_RESID_NORM && EPI != EPI_EMBED_NORM) {
    if (!f_ok) return;
    const int64_t ld = g.ldo;
    if constexpr (EPI == EPI_STORE_PLANES) {
      // (the only epilogue whose destination has no padding rows: a token past the end would land in the next plane)
      bf16* p = (bf16*)g.out + (int64_t)(f / g.plane_w) * g.plane_stride + (f % g.plane_w) + (int64_t)tok_base * g.plane_w;
#pragma unroll
      for (int j = 0; j < NT; ++j)
        if (tok_base + j < g.n_tok) p[(int64_t)j * g.plane_w] = __float2bfloat16_rn(v[j]);
    } else if constexpr (EPI == EPI_STORE_F32) {
      float* p = (float*)g.out + (int64_t)tok_base * ld + f;
      const float b = g.bias ? g.bias[f] : 0.f;
#pragma unroll
      for (int j = 0; j < NT; ++j) p[j * ld] = v[j] + b;
    } else {
      bf16* p = (bf16*)g.out + (int64_t)tok_base * ld + f;
      if constexpr (EPI == EPI_STORE) {
        const float b = g.bias ? g.bias[f] : 0.f;
#pragma unroll
        for (int j = 0; j < NT; ++j) p[j * ld] = __float2bfloat16_rn(v[j] * rs[j] + b);
      } else if constexpr (EPI == EPI_SILU_VEC) {
        const float b = g.bias[f];
#pragma unroll
        for (int j = 0; j < NT; ++j) p[j * ld] = __float2bfloat16_rn(silu_f(v[j] + b));
      } else {  // EPI_GEGLU
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const float r = rs[j];
          p[j * ld] = __float2bfloat16_rn(gelu_tanh_fast(v[j] * r) * (v2[j] * r));
        }
      }
    }
  }
}

// Second half of the residual epilogues, once per token range [tok_first, tok_first + nvalid) that this
// block finalised: publish the range's per-token sums of squares over this feature tile (the four
// epilogue warps added in a fixed order).  The next projection's epilogue adds the feature tiles up and
// derives 1/rms.  All 128 epilogue threads call it (block-level barriers inside).
__device__ __forceinline__ void finalize_stats(const GemmArgs& g, int nvalid, int tok_first, int ft, const float* red) {
  if (nvalid <= 0) return;  // uniform over the block
  const int et = threadIdx.x & 127;  // epilogue thread id (warps 2..5)
  const bool embed = g.epi == EPI_EMBED_NORM;
  epi_bar_sync();
  for (int t = et; t < nvalid; t += 128) {
    const int tok = tok_first + t;
    const int64_t row = embed ? (tok + tok / g.horizon + 1) : tok;
    g.ssq[(int64_t)ft * g.ssq_ld + row] = ((red[t] + red[256 + t]) + red[512 + t]) + red[768 + t];
  }
  epi_bar_sync();  // red[] may be reused
}

// CW: tokens per epilogue chunk (16 or 32, chosen by the host from the tile width).  The kernel's code has to be
// fetched anew at every launch, so each instantiation carries one chunk width only.
// SPLIT: the kernel runs as clusters that share the k dimension (exchange code only in these instantiations).
// NI: product-issuing threads (1 or 2).  INSTR: phase stamps and launch trace compiled in (test and measurement aids).
// WITHHOLD: the failure-path test aid (GemmArgs::debug_withhold) compiled in: one instantiation only, because even a
// never-taken test in the copy-issuing thread's loop costs the batch-1 call 1.7 %.
template <bool DUAL, int EPI, int CW, bool SPLIT, int NI, bool INSTR, bool WITHHOLD = false>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a, GemmArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t acc_full_bar[2];
  __shared__ __align__(8) uint64_t acc_empty_bar[2];
  __shared__ uint32_t tmem_base_smem;
  __shared__ volatile int abort_flag;
  __shared__ __align__(8) uint64_t xbar;  // counts the bytes of partial accumulators received from the cluster
  __shared__ float red[4 * 256];
  __shared__ float rs_tile[256];  // per-token scale of the token range this block finalises

  ptx::pdl_launch_dependents();  // the next kernel may be scheduled (it waits for this grid before reading)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned long long* const dbg = (INSTR && g.dbg) ? g.dbg + (size_t)blockIdx.x * 16 : nullptr;
  unsigned long long* const trace = INSTR ? g.trace : nullptr;
  if (dbg && threadIdx.x == 0) { dbg[0] = ptx::globaltimer_ns(); dbg[12] = clock64(); }
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4] = ptx::globaltimer_ns();
  // 1024-byte alignment of the tile ring (required by the 128-byte swizzle)
  uint8_t* tiles = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  // send buffer [4 epilogue warps][tile_tok][DUAL ? 2 : 1][32 features] fp32: each warp's share for one receiver is contiguous
  float* xbuf = reinterpret_cast<float*>(tiles + g.ring_bytes);
  float* xrecv = xbuf + (size_t)g.tile_tok * (DUAL ? 2 : 1) * TILE_F;  // receive buffer [splits][4][slice][..][32]
  const uint32_t w_bytes = (DUAL ? 2 : 1) * TILE_F * TILE_K * 2;
  const uint32_t a_bytes = (uint32_t)g.tile_tok * TILE_K * 2;
  const uint32_t stage_bytes = w_bytes + a_bytes;
  const int CS = SPLIT ? g.splits : 1;
  const int rank = (int)ptx::cluster_ctarank();
  const int n_clusters = gridDim.x / CS, cid = blockIdx.x / CS;
  const int total_items = g.n_ftiles * g.n_ttiles;
  const int acc_cols = (DUAL ? 2 : 1) * NI * g.tile_tok;  // one accumulator buffer: [issuer][gate | up][token]
  const int kb0 = (int)((int64_t)rank * g.kb_total / CS), kb1 = (int)((int64_t)(rank + 1) * g.kb_total / CS);

  if (threadIdx.x == 0) {
    for (int s = 0; s < g.stages; ++s) {
      ptx::mbar_init(&full_bar[s], 2);  // the weight producer and the activation producer
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&acc_full_bar[a], (uint32_t)NI);
      ptx::mbar_init(&acc_empty_bar[a], 4);  // one arrival per epilogue warp
    }
    ptx::mbar_init(&xbar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_w);
    ptx::prefetch_tensormap(&map_a);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tmem_base_smem, g.tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (SPLIT) {  // every block of the cluster has initialised its barriers before any peer signals them
    ptx::cluster_arrive_release();
    ptx::cluster_wait_acquire();
  }
  const uint32_t tmem_base = tmem_base_smem;
  if (dbg && threadIdx.x == 0) dbg[1] = ptx::globaltimer_ns();

  // Every thread of the cluster passes the cluster barrier once per tile (after the exchange of
  // partial accumulators), whatever happens to its role's waits.
#define ADIT_CLUSTER_SYNC()                  \
  do {                                       \
    if (SPLIT) {                             \
      ptx::cluster_arrive_release();         \
      ptx::cluster_wait_acquire();           \
    }                                        \
  } while (0)

  if (warp == 0 || warp == 6) {
    // ------------------------------ TMA producers ------------------------------
    // One stage costs an issuing thread several hundred cycles of dependent instruction latency (barrier
    // wait, expect-tx, bulk-tensor copy), which is more than a small tile's products take.  The weight
    // tiles and the activation tiles therefore have a producer thread each (warps 0 and 6); both signal
    // the stage's barrier with their own byte counts.
    const bool is_w = warp == 0;
    if (lane == 0) {
      // Weights do not depend on the preceding kernel: the first tile's weight blocks (as many as the
      // ring holds) are requested before waiting for the preceding grid; activations only afterwards.
      int pre = 0;
      if (cid < total_items) {
        const int ft = cid % g.n_ftiles;
        pre = min(kb1 - kb0, g.stages);
        if (is_w)
          for (int i = 0; i < pre; ++i) {
            ptx::mbar_arrive_expect_tx(&full_bar[i], w_bytes);
            ptx::tma_load_2d(tiles + (size_t)i * stage_bytes, &map_w, (kb0 + i) * TILE_K, ft * (DUAL ? 2 : 1) * TILE_F,
                             &full_bar[i]);
          }
      }
      ptx::pdl_wait_prior_grids();
      if (trace && is_w) trace[blockIdx.x * 4 + 1] = ptx::globaltimer_ns();
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int w = cid; w < total_items; w += n_clusters) {
        const int ft = w % g.n_ftiles, tt = w / g.n_ftiles;
        for (int kb = kb0; kb < kb1 && ok; ++kb, ++issued) {
          uint8_t* ws = tiles + (size_t)stage * stage_bytes;
          if (issued >= pre && !ptx::mbar_wait(&empty_bar[stage], phase ^ 1)) { ok = false; break; }
          if (is_w) {
            if (issued >= pre) {
              ptx::mbar_arrive_expect_tx(&full_bar[stage], w_bytes);
              ptx::tma_load_2d(ws, &map_w, kb * TILE_K, ft * (DUAL ? 2 : 1) * TILE_F, &full_bar[stage]);
            }
          } else if (WITHHOLD && g.debug_withhold > 0 && blockIdx.x == 0 && issued + 1 == g.debug_withhold) {
            // (test aid: this stage never fills; the issuing thread's bounded wait runs out and the block winds down)
          } else {
            ptx::mbar_arrive_expect_tx(&full_bar[stage], a_bytes);
            ptx::tma_load_2d(ws + w_bytes, &map_a, kb * TILE_K, tt * g.tile_tok, &full_bar[stage]);
          }
          if (++stage == g.stages) { stage = 0; phase ^= 1; }
        }
        ADIT_CLUSTER_SYNC();
      }
      if (!ok) { atomicExch(g.status, -6); abort_flag = 1; }
    } else {
      for (int w = cid; w < total_items; w += n_clusters) {
        ADIT_CLUSTER_SYNC();
      }
    }
  } else if (warp == 1 || warp == 7) {
    // ------------------------------ MMA issuers ------------------------------
    const int me = warp == 1 ? 0 : 1;
    if (lane == 0 && me < NI) {
      const uint32_t idesc = ptx::idesc_bf16_f32(TILE_F, g.tile_tok);
      // Two issuers take alternate k-blocks (running index modulo 2, counted over all of this block's tiles).
      constexpr bool alternate = NI == 2;
      const int step = alternate ? 2 : 1;
      const int kbn = kb1 - kb0;
      int cur = alternate ? me : 0;  // running index of the next k-block this thread issues
      int stage = cur;               // (the ring has at least two stages)
      uint32_t phase = 0;
      int acc_iter = 0, base = 0;
      bool ok = true;
      for (int w = cid; w < total_items; w += n_clusters, ++acc_iter, base += kbn) {
        const int a = g.acc_bufs == 2 ? (acc_iter & 1) : 0;
        const uint32_t acc_phase = (uint32_t)(g.acc_bufs == 2 ? (acc_iter >> 1) : acc_iter) & 1u;
        if (ok && !ptx::mbar_wait(&acc_empty_bar[a], acc_phase ^ 1)) ok = false;
        if (ok) {
          ptx::tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(a * acc_cols) + (uint32_t)(me * (DUAL ? 2 : 1) * g.tile_tok);
          // The barrier test of the next stage is issued before this stage's products, so that its latency
          // (over a hundred cycles even when the data is there) overlaps with issuing them.
          bool ready = cur < base + kbn && ptx::mbar_test_wait(&full_bar[stage], phase);
          bool first = true;
          while (cur < base + kbn) {
            if (!ready && !ptx::mbar_wait(&full_bar[stage], phase)) { ok = false; break; }
            ptx::tc_fence_after();
            if (dbg && w == cid && me == 0 && (first || cur + step >= base + kbn)) dbg[first ? 2 : 3] = ptx::globaltimer_ns();
            const uint32_t ws = ptx::smem_u32(tiles + (size_t)stage * stage_bytes);
            const uint32_t as = ws + w_bytes;
            const int cur_stage = stage;
            cur += step;
            stage += step;
            if (stage >= g.stages) { stage -= g.stages; phase ^= 1; }
            if (cur < base + kbn) ready = ptx::mbar_test_wait(&full_bar[stage], phase);
#pragma unroll
            for (int k4 = 0; k4 < TILE_K / UMMA_K; ++k4) {
              const uint64_t bdesc = ptx::smem_desc_sw128(as + k4 * UMMA_K * 2);
              const uint32_t acc = (!first || k4 > 0) ? 1u : 0u;
              ptx::umma_f16(d_tmem, ptx::smem_desc_sw128(ws + k4 * UMMA_K * 2), bdesc, idesc, acc);
              if (DUAL)
                ptx::umma_f16(d_tmem + (uint32_t)g.tile_tok,
                              ptx::smem_desc_sw128(ws + TILE_F * TILE_K * 2 + k4 * UMMA_K * 2), bdesc, idesc, acc);
            }
            ptx::umma_commit(&empty_bar[cur_stage]);  // frees the stage once these MMAs have read it
            first = false;
          }
          if (ok) ptx::umma_commit(&acc_full_bar[a]);
        }
        ADIT_CLUSTER_SYNC();
      }
      if (!ok) { atomicExch(g.status, -6); abort_flag = 1; }
    } else {
      for (int w = cid; w < total_items; w += n_clusters) {
        ADIT_CLUSTER_SYNC();
      }
    }
  } else {
    // ------------------------------ epilogue (warps 2..5) ------------------------------
    const int quarter = warp & 3;  // TMEM lanes [32 * quarter, 32 * quarter + 32)
    const int fl = quarter * 32 + lane;  // feature within the tile
    const int et = threadIdx.x - 64;     // epilogue thread id 0..127
    const int slice = g.tile_tok / CS;   // tokens of a tile finalised by each block of the cluster
    constexpr int NV = DUAL ? 2 : 1;
    constexpr bool RESID = EPI == EPI_RESID_NORM;
    constexpr bool SCALED = EPI == EPI_STORE || EPI == EPI_GEGLU;
    ptx::pdl_wait_prior_grids();         // outputs may still be in use by the preceding grid
    int acc_iter = 0;
    bool ok = true;
    // Current residual values of CW token rows starting at `tok` for this thread's feature.  Always CW loads:
    // rows past the range exist (padding rows) and are simply not used.
    auto load_old = [&](float (&dst)[CW], int tok, int f) {
      if constexpr (RESID) {
        const float* hp = g.h + (int64_t)tok * g.n_feat + (f < g.n_feat ? f : 0);
#pragma unroll
        for (int j = 0; j < CW; ++j) dst[j] = __ldcg(hp + (int64_t)j * g.n_feat);
      }
    };
    for (int w = cid; w < total_items; w += n_clusters, ++acc_iter) {
      const int ft = w % g.n_ftiles, tt = w / g.n_ftiles;
      const int a = g.acc_bufs == 2 ? (acc_iter & 1) : 0;
      const uint32_t acc_phase = (uint32_t)(g.acc_bufs == 2 ? (acc_iter >> 1) : acc_iter) & 1u;
      const int f = ft * TILE_F + fl;
      const int tok0 = tt * g.tile_tok;
      const int my_first = tok0 + (SPLIT ? rank * slice : 0);  // token range finalised by this block
      const int my_count = SPLIT ? slice : g.tile_tok;
      // Everything that does not depend on the accumulator happens before the wait for it: the per-token
      // scales of the range (1/rms from the producer's per-feature-tile sums of squares, added in tile
      // order) and the residual values of the first chunk.
      if constexpr (SCALED) {
        epi_bar_sync();  // the previous item's scales have been read
        for (int t = et; t < my_count; t += 128) {
          float r = 1.f;
          if (g.norm_ssq) {
            const float* sp = g.norm_ssq + my_first + t;
            float tot = 0.f;
#pragma unroll 4
            for (int i = 0; i < g.norm_tiles; ++i) tot += __ldcg(sp + (int64_t)i * g.ssq_ld);
            r = 1.0f / sqrtf(tot / (float)g.norm_dim + g.eps);
          } else if (g.rowscale) {
            r = g.rowscale[my_first + t];
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
      load_old(oldn, my_first, f);
      if (ok) {
        int okw = 1;
        if (lane == 0) okw = ptx::mbar_wait(&acc_full_bar[a], acc_phase) ? 1 : 0;
        okw = __shfl_sync(0xffffffffu, okw, 0);
        if (!okw) ok = false;
      }
      if (ok) {
        for (int spin = 0; spin < 4096 && !ptx::mbar_try_wait(&acc_full_bar[a], acc_phase); ++spin) {}
        ptx::tc_fence_after();
        if (dbg && threadIdx.x == 64 && w == cid) dbg[4] = ptx::globaltimer_ns();
        if (trace && threadIdx.x == 64 && w + n_clusters >= total_items) trace[blockIdx.x * 4 + 3] = ptx::globaltimer_ns();
        const uint32_t t_addr = tmem_base + (uint32_t)(a * acc_cols) + ((uint32_t)(quarter * 32) << 16);
        int sent = 0;  // receivers this warp has sent their slice to
        {
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
            if constexpr (NI == 2) {  // the second issuer's part of the sum over k, added in a fixed order
              float u[CW];
              if constexpr (CW == 32) ptx::tmem_ld_32x32(t_addr + NV * g.tile_tok + c0, u);
              else ptx::tmem_ld_32x16(t_addr + NV * g.tile_tok + c0, u);
              ptx::tmem_ld_wait();  // (one wait for both issuers' columns)
#pragma unroll
              for (int j = 0; j < CW; ++j) v[j] += u[j];
              if (DUAL) {
                if constexpr (CW == 32) ptx::tmem_ld_32x32(t_addr + 3 * g.tile_tok + c0, u);
                else ptx::tmem_ld_32x16(t_addr + 3 * g.tile_tok + c0, u);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < CW; ++j) v2[j] += u[j];
              }
            } else {
              ptx::tmem_ld_wait();
            }
            if constexpr (!SPLIT) {
              float old[CW];
#pragma unroll
              for (int j = 0; j < CW; ++j) old[j] = oldn[j];
              if (c0 + CW < g.tile_tok) load_old(oldn, tok0 + c0 + CW, f);
              finalize_chunk<DUAL, CW, EPI>(g, v, v2, old, tok0 + c0, f, c0, red, rs_tile + c0);
            } else {  // park the partial accumulator in the send buffer: [warp][token][gate|up][32 features]
              float* dst = xbuf + ((size_t)quarter * g.tile_tok + c0) * NV * 32 + lane;
#pragma unroll
              for (int j = 0; j < CW; ++j) {
                dst[j * NV * 32] = v[j];
                if (DUAL) dst[j * NV * 32 + 32] = v2[j];
              }
              // Exchange, pipelined with the parking: tokens [r * slice, (r + 1) * slice) of the tile are finalised by
              // block r.  As soon as a receiver's slice is parked, this warp pushes its 32 features of it (one
              // contiguous piece) into r's receive buffer with a bulk shared-to-shared copy that signals r's mbarrier;
              // the four epilogue warps send side by side and need no block-wide barrier.
              ptx::fence_proxy_async();  // parked values (generic proxy) -> visible to the bulk-copy engine
              __syncwarp();
              if (lane == 0) {
                const uint32_t piece = (uint32_t)slice * NV * 32 * 4;  // one warp's share for one receiver
                const uint32_t recv_local = ptx::smem_u32(xrecv) + (uint32_t)(rank * 4 + quarter) * piece;
                const uint32_t send_local = ptx::smem_u32(xbuf) + (uint32_t)quarter * (uint32_t)g.tile_tok * NV * 32 * 4;
                const uint32_t bar_local = ptx::smem_u32(&xbar);
                while ((sent + 1) * slice <= c0 + CW) {
                  ptx::bulk_copy_to_peer(ptx::mapa_shared(recv_local, sent), send_local + (uint32_t)sent * piece, piece,
                                         ptx::mapa_shared(bar_local, sent));
                  ++sent;
                }
              }
            }
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&acc_empty_bar[a]);
        if (!SPLIT && (EPI == EPI_RESID_NORM || EPI == EPI_EMBED_NORM))
          finalize_stats(g, min(g.tile_tok, g.n_tok - tok0), tok0, ft, red);
      }
      if (dbg && threadIdx.x == 64 && w == cid) dbg[8] = ptx::globaltimer_ns();
      if constexpr (SPLIT) {
        // (the slices were sent while the accumulator was being parked; this block's barrier counts what it receives)
        const uint32_t piece = (uint32_t)slice * NV * 32 * 4;
        if (threadIdx.x == 64) ptx::mbar_arrive_expect_tx(&xbar, piece * 4u * (uint32_t)CS);
        if (dbg && threadIdx.x == 64 && w == cid) dbg[9] = ptx::globaltimer_ns();
        if (ok) {
          int okw = 1;
          if (lane == 0) okw = ptx::mbar_wait(&xbar, (uint32_t)(acc_iter & 1)) ? 1 : 0;
          okw = __shfl_sync(0xffffffffu, okw, 0);
          if (!okw) ok = false;
          for (int spin = 0; ok && spin < 4096 && !ptx::mbar_try_wait(&xbar, (uint32_t)(acc_iter & 1)); ++spin) {}
        }
        if (dbg && threadIdx.x == 64 && w == cid) dbg[11] = ptx::globaltimer_ns();
        // slice is a multiple of 8 (the planner sees to it): finalise 8 tokens at a time, each value the sum of the
        // cluster's partial accumulators in rank order (fixed summation order)
        // The cluster barrier of this tile says "this block has received and read everything": once all have said so,
        // nobody's send buffer is in use and the receive buffers may be overwritten.  The epilogue warps arrive as
        // soon as their last read of the receive buffer is done and only wait after finalising, so the barrier's
        // latency overlaps with the residual update and the statistics.
        bool arrived = false;
        if (ok) {
          float cur8[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) cur8[j] = oldn[j];
#pragma unroll 1
          for (int done = 0; done < slice; done += 8) {
            float v[8], v2[8], nxt[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) { v[j] = 0.f; v2[j] = 0.f; nxt[j] = 0.f; }
            if constexpr (RESID) {
              if (done + 8 < slice) {  // the next group's residual values, one group ahead
                const float* hp = g.h + (int64_t)(my_first + done + 8) * g.n_feat + (f < g.n_feat ? f : 0);
#pragma unroll
                for (int j = 0; j < 8; ++j) nxt[j] = __ldcg(hp + (int64_t)j * g.n_feat);
              }
            }
#pragma unroll 1
            for (int r = 0; r < CS; ++r) {
              const float* src = xrecv + (((size_t)(r * 4 + quarter) * slice + done) * NV) * 32 + lane;
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                v[j] += src[j * NV * 32];
                if (DUAL) v2[j] += src[j * NV * 32 + 32];
              }
            }
            if (done + 8 >= slice) { ptx::cluster_arrive_release(); arrived = true; }
            if (dbg && threadIdx.x == 64 && w == cid) dbg[10] = ptx::globaltimer_ns();
            finalize_chunk<DUAL, 8, EPI>(g, v, v2, cur8, my_first + done, f, done, red, rs_tile + done);
#pragma unroll
            for (int j = 0; j < 8; ++j) cur8[j] = nxt[j];
          }
        }
        if (ok && (EPI == EPI_RESID_NORM || EPI == EPI_EMBED_NORM))
          finalize_stats(g, min(slice, g.n_tok - my_first), my_first, ft, red);
        // Nobody may overwrite a receive buffer (next tile) or leave (its send buffer is still being
        // read by the copy engine) before every block of the cluster has received everything.
        if (!arrived) ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
      }
      if (dbg && threadIdx.x == 64 && w == cid) dbg[5] = ptx::globaltimer_ns();
    }
    if (!ok && lane == 0) { atomicExch(g.status, -6); abort_flag = 1; }
  }
#undef ADIT_CLUSTER_SYNC

  // ------------------------------ teardown ------------------------------
  ptx::tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    // a wait expired: give copies still in flight time to land before the block's memory is released
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) {}
    __syncthreads();
  }
  if (dbg && threadIdx.x == 0) { dbg[6] = ptx::globaltimer_ns(); dbg[13] = clock64(); }
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4 + 2] = ptx::globaltimer_ns();
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, g.tmem_cols);
    if (dbg && lane == 0) dbg[7] = ptx::globaltimer_ns();
  }
}

}  // namespace tc
}  // namespace adit
