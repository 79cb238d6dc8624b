// The whole denoising loop of a small batch (at most 64 suffix tokens in total) as ONE persistent kernel.
//
// At batch 1 an Euler step streams 640 MB of weights through 5 data-dependent phases per layer; run as one
// kernel per phase, every phase boundary stops the weight stream and pays a launch hand-off.  Here the grid
// is a fixed set of thread-block clusters (8 blocks each, one block per SM, at most sm_budget blocks) that
// stays resident for all K steps x L layers:
//
//   * weights: every block walks a static list of 128-feature x 64-k weight tiles (its share of every
//     projection of every layer) and keeps a ring of them in flight with TMA; the producer thread is throttled
//     only by ring space, never by a phase boundary, so the next phase's weights are in shared memory before
//     its activations exist;
//   * phases ("levels") are separated by counters in global memory: a block adds 1 with release semantics
//     when its part of a level is stored, the consumers poll with acquire semantics (one polling thread
//     per block), bounded by a time limit;
//   * a projection level is cut into cluster units: nf feature tiles x ks k-slices = 8 blocks.  Each block
//     multiplies its k-slice (tcgen05, accumulator in tensor memory: lane = feature, column = token), writes the
//     partial sums to a per-cluster scratch in global memory (it stays in L2), signals the cluster's blocks through
//     their mbarriers, and the block that owns a token adds the ks partials in slice order - bitwise reproducible,
//     independent of the grid size - and runs the fused epilogue (1/rms scale, GeGLU, residual + bf16 copy + sums of
//     squares for the next norm);
//   * an attention level is cut into units of (request, kv head, 128 query rows); the 8 blocks of a cluster
//     take 8 ranges of 64-key blocks (prefix keys padded to a multiple of 64 with masked, zero-filled rows,
//     then the suffix keys), K/V and Q tiles come in by TMA (prefix blocks before the level's flag: they do
//     not depend on the step), and the split results are merged inside the cluster the same way: every row's
//     unnormalised partial goes to the scratch, the block that owns the row combines the 8 splits in fixed order;
//   * the per-step element-wise work (first embedding layer, read-out + Euler update) are levels of their
//     own, spread over all blocks.
//
// Warp roles (256 threads): 0 = weight producer / K,V loader, 1 = flag poller + activation / Q loader,
// 2 = MMA issuer (projections, Q K^T), 3 = TMEM owner + P V issuer, 4-7 = epilogue / softmax.
// Shared memory (227 KB): projections see [10 weight slots | 8 activation slots],
// attention sees [K ring | P | V ring | Q] in the same bytes; a block never runs both at once, and the
// weight producer drains its ring before an attention unit.  Every wait is bounded.
#pragma once
#include "attention.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "ptx.cuh"

namespace adit {
namespace loop {

constexpr int CS = 8;           // blocks per cluster
constexpr int TOK = 64;         // token tile (MMA N); the path serves at most this many suffix tokens
constexpr int NSW = 10;         // weight slots of 128 features x 64 k (16 KB)
constexpr int W_SLOT = 16384;
constexpr int NSA = 8;          // activation slots of 64 tokens x 64 k (8 KB)
constexpr int A_SLOT = 8192;
constexpr int OFF_W = 0;
constexpr int OFF_A = NSW * W_SLOT;            // 160 KB
constexpr int POOL = OFF_A + NSA * A_SLOT;     // 224 KB
// attention view of the same pool
constexpr int OFF_K = 0;                       // 2 stages of 64 keys x dh (<= 64 KB)
constexpr int OFF_P = 65536;                   // 2 x [128 rows][64 keys] bf16 (32 KB)
constexpr int OFF_V = 98304;                   // 2 stages (<= 64 KB)
constexpr int OFF_Q = OFF_A;                   // 128 rows x dh (<= 64 KB)
// Partial sums of a cluster travel through global memory (L2): per cluster, per source block either
// [gate | up][64 tokens][128 features] fp32 or [128 rows][dh] bf16 + [128] (max, sum) pairs.  (Distributed shared
// memory moves about 13 GB/s per block on this part; the same bytes through L2 take a fraction of that time.)
constexpr int XS_BLOCK_BYTES = 2 * TOK * 128 * 4;                  // 64 KB per source block
constexpr int XS_ML_OFF = CS * XS_BLOCK_BYTES;                     // (max, sum) pairs after the partials
constexpr int XS_CLUSTER_BYTES = XS_ML_OFF + CS * 128 * 8;         // 520 KB per cluster
constexpr int MISC_BYTES = 3072;
constexpr int SMEM_BYTES = POOL + MISC_BYTES;  // 232448 = the per-block maximum
constexpr int THREADS = 256;
constexpr int MAXB = 4;                        // requests per call on this path

enum : int { LV_EMBED_IN = 0, LV_W2, LV_QKV, LV_ATT, LV_O, LV_GU, LV_DOWN, LV_FINAL, LV_COUNT };
enum : int { G_W2 = 0, G_QKV, G_O, G_GU, G_DOWN, G_COUNT };
// tensor maps in device memory: fixed ones first, then four per layer (qkv, o, gate/up, down)
enum : int { MAP_W2 = 0, MAP_A_EZ, MAP_A_HB, MAP_A_ATT, MAP_A_MLP, MAP_Q3D, MAP_KV2D, MAP_LAYER0 };
enum : int { LEPI_STORE = 0, LEPI_GEGLU, LEPI_RESID, LEPI_EMBED };

struct GemmLv {
  int n_ftiles;  // output tiles of 128 features (gate/up: pairs of tiles)
  int kb_total;  // K / 64
  int ks;        // k-slices per feature tile = partial sums per output element (8, 4 or 2)
  int nf;        // feature tiles per cluster unit = 8 / ks
  int kbn;       // k-blocks per slice
  int units;     // cluster units per level
  int dual;      // gate/up pair
  int epi;       // LEPI_*
  int map_a;     // activation tensor map
  int ldo;       // leading dimension of the bf16 output (STORE, GEGLU)
};

struct LoopParams {
  alignas(64) CUtensorMap pk[MAXB];  // per request: prefix cache as (channel, row < prefix_len, plane)
  alignas(64) CUtensorMap kv2d;      // this step's K/V rows of the qkv workspace, row extent = the call's token count
  const CUtensorMap* maps;           // device array, see MAP_*
  int plen[MAXB];
  GemmLv g[G_COUNT];
  int L, K, D, F, n_q_heads, n_kv_heads, n_tok, horizon, A, B, M, Ma;
  int n_clusters, n_row_tiles, att_units, ssq_ld, n_dtiles;
  float scale_log2, eps, dt;
  float *x, *h, *ssq, *out;
  bf16 *hb, *qkv, *att, *mlp, *ez;
  const float *Wfold, *bfold, *ctime, *hs, *ssq_state, *Wout, *bout, *b2;
  const bf16* hsb;
  uint8_t* xscratch;   // n_clusters x XS_CLUSTER_BYTES
  uint32_t* counters;  // [LV_COUNT] level counters, [LV_COUNT] abort word; zeroed before every call
  int* status;         // host-visible status word
  unsigned long long timeout_ns;
  int state_mask;        // variant: the state token attends to the prefix and itself only
  int debug_skip_level;  // test aid: the level type whose first flag increment of block 0 is withheld (-1: none)
  unsigned long long* trace;  // optional [level][block][8] timestamps
};

struct Misc {
  uint64_t wfull[NSW], wempty[NSW], afull[NSA], aempty[NSA];
  uint64_t acc_full, unit_done, level_go, xfull, xfree;
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], s_empty[2], p_full[2], pv_done[2];
  uint64_t q_full, epi_bar;
  uint32_t tmem_base;
  volatile int abort;
  volatile int level_seen;  // participating levels whose dependency the polling thread has observed
  volatile int units_done;  // units this block's epilogue warps have finished
  float red[4];
};
static_assert(sizeof(Misc) <= MISC_BYTES, "misc region too small");

struct Ctx {
  const LoopParams* p;
  Misc* ms;
  uint8_t* pool;
  uint32_t tmem;
  int cid, rank, n_cta, cta;
};

// ---- bounded waits ------------------------------------------------------------------------------
__device__ __forceinline__ bool gave_up(const Ctx& c, uint64_t t0) {
  if (c.ms->abort) return true;
  if (*(volatile uint32_t*)(c.p->counters + LV_COUNT) != 0u) return true;
  return ptx::globaltimer_ns() - t0 > c.p->timeout_ns;
}
__device__ __noinline__ void fail(const Ctx& c) {
  atomicExch(c.p->status, -6);
  atomicExch(c.p->counters + LV_COUNT, 1u);
  c.ms->abort = 1;
}
// Waiting must not starve the warps that work: a tight polling loop on a shared-memory barrier fills the memory
// pipeline that the epilogue's loads and stores and the tensor-core issue go through.  Waits that are expected to be
// long (ring space, the end of a unit) use the suspending try_wait; waits on the critical path of a level poll the
// non-blocking test with a short sleep in between.
__device__ __forceinline__ void nap(unsigned ns) { asm volatile("nanosleep.u32 %0;" ::"r"(ns)); }
template <bool CRITICAL = true>
__device__ __forceinline__ bool bwait(const Ctx& c, uint64_t* bar, uint32_t parity) {
  if (ptx::mbar_test_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 512; ++i) {
      if (CRITICAL) {
        nap(20);
        if (ptx::mbar_test_wait(bar, parity)) return true;
      } else {
        if (ptx::mbar_try_wait(bar, parity)) return true;
      }
    }
    if (gave_up(c, t0)) return false;
  }
}
// Whole-warp wait: lane 0 waits, the others rejoin at the shuffle.
__device__ __forceinline__ bool warp_wait(const Ctx& c, uint64_t* bar, uint32_t parity) {
  int okw = 1;
  if ((threadIdx.x & 31) == 0) okw = bwait<true>(c, bar, parity) ? 1 : 0;
  okw = __shfl_sync(0xffffffffu, okw, 0);
  if (!okw) return false;
  // (every lane performs the acquiring test itself; the phase is complete, so this does not spin)
  while (!ptx::mbar_test_wait(bar, parity)) {}
  return true;
}
// Wait on a count in shared memory that only grows.  A thread that runs ahead of the others by several phases
// (the weight producer) cannot wait on an mbarrier parity, which only tells neighbouring phases apart.
__device__ __forceinline__ bool wait_count(const Ctx& c, const volatile int* v, int target) {
  if (*v >= target) { __threadfence_block(); return true; }
  const uint64_t t0 = ptx::globaltimer_ns();
  int spins = 0;
  while (*v < target) {
    nap(40);
    if ((++spins & 255) == 0 && gave_up(c, t0)) return false;
  }
  __threadfence_block();
  return true;
}
__device__ __forceinline__ bool poll_counter(const Ctx& c, const uint32_t* cnt, uint32_t target) {
  // relaxed polls (an acquire per poll costs a fence each time), one acquire fence once the count is there
  bool seen = ptx::ld_relaxed_gpu(cnt) >= target;
  if (!seen) {
    const uint64_t t0 = ptx::globaltimer_ns();
    while (!seen) {
#pragma unroll 1
      for (int i = 0; i < 64 && !seen; ++i) seen = ptx::ld_relaxed_gpu(cnt) >= target;
      if (!seen && gave_up(c, t0)) return false;
    }
  }
  ptx::fence_acq_rel_gpu();
  return true;
}
// Barrier of the four epilogue warps on an mbarrier, so that it is bounded like every other wait: a warp that gave
// up never arrives and the others leave through the time limit / abort flag instead of hanging in bar.sync.
__device__ __forceinline__ bool epi_sync(const Ctx& c, int& nsync) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(&c.ms->epi_bar);
  const bool r = warp_wait(c, &c.ms->epi_bar, (uint32_t)nsync & 1u);
  ++nsync;
  return r;
}

// ---- the static schedule ------------------------------------------------------------------------
struct Lv {
  int type, k, l;
  int units;   // cluster units (0: a level spread over all blocks)
  int off;     // rotation: unit u runs on cluster (u + off) % n_clusters
  int dep;     // counter this level waits for (-1: none)
  uint32_t dep_target;
  int seq;     // running index of the level within the call
};
__device__ __forceinline__ int level_gemm(int type) { return type == LV_W2 ? G_W2 : type == LV_QKV ? G_QKV : type == LV_O ? G_O : type == LV_GU ? G_GU : G_DOWN; }

template <typename F>
__device__ __forceinline__ void walk_levels(const LoopParams& p, F&& f) {
  const int C = p.n_clusters;
  const uint32_t ncta = (uint32_t)C * CS;
  int off = 0, seq = 0;
  for (int k = 0; k < p.K; ++k) {
    for (int j = -2; j <= 5 * p.L; ++j, ++seq) {
      Lv lv;
      lv.k = k; lv.l = 0; lv.off = off; lv.seq = seq; lv.units = 0;
      if (j == -2) {
        lv.type = LV_EMBED_IN; lv.dep = k ? LV_FINAL : -1; lv.dep_target = (uint32_t)k * ncta;
      } else if (j == -1) {
        lv.type = LV_W2; lv.units = p.g[G_W2].units; lv.dep = LV_EMBED_IN; lv.dep_target = (uint32_t)(k + 1) * ncta;
      } else if (j == 5 * p.L) {
        lv.type = LV_FINAL; lv.dep = LV_DOWN; lv.dep_target = (uint32_t)((k + 1) * p.L) * (uint32_t)(p.g[G_DOWN].units * CS);
      } else {
        const int l = j / 5, t = j - 5 * l;
        const uint32_t inst = (uint32_t)(k * p.L + l);
        lv.l = l;
        if (t == 0) {
          lv.type = LV_QKV; lv.units = p.g[G_QKV].units;
          if (l == 0) { lv.dep = LV_W2; lv.dep_target = (uint32_t)(k + 1) * (uint32_t)(p.g[G_W2].units * CS); }
          else { lv.dep = LV_DOWN; lv.dep_target = inst * (uint32_t)(p.g[G_DOWN].units * CS); }
        } else if (t == 1) {
          lv.type = LV_ATT; lv.units = p.att_units; lv.dep = LV_QKV; lv.dep_target = (inst + 1) * (uint32_t)(p.g[G_QKV].units * CS);
        } else if (t == 2) {
          lv.type = LV_O; lv.units = p.g[G_O].units; lv.dep = LV_ATT; lv.dep_target = (inst + 1) * (uint32_t)(p.att_units * CS);
        } else if (t == 3) {
          lv.type = LV_GU; lv.units = p.g[G_GU].units; lv.dep = LV_O; lv.dep_target = (inst + 1) * (uint32_t)(p.g[G_O].units * CS);
        } else {
          lv.type = LV_DOWN; lv.units = p.g[G_DOWN].units; lv.dep = LV_GU; lv.dep_target = (inst + 1) * (uint32_t)(p.g[G_GU].units * CS);
        }
      }
      f(lv);
      off = (off + lv.units) % C;
    }
  }
}
// First unit of level lv that runs on cluster cid (units cid_first, cid_first + C, ...).
__device__ __forceinline__ int first_unit(const Lv& lv, int cid, int C) { int u = cid - lv.off; return u < 0 ? u + C : u; }
__device__ __forceinline__ bool participates(const Lv& lv, int cid, int C) { return lv.units == 0 || first_unit(lv, cid, C) < lv.units; }

struct GemmUnit { int ft, sl, grp; bool valid; };
__device__ __forceinline__ GemmUnit gemm_unit(const GemmLv& g, int u, int rank) {
  GemmUnit r;
  r.grp = rank / g.ks; r.sl = rank - r.grp * g.ks; r.ft = u * g.nf + r.grp; r.valid = r.ft < g.n_ftiles;
  return r;
}
struct AttUnit { int b, kvh, rt, plen, npb, nkb, kb0, kb1, tok0; };
__device__ __forceinline__ AttUnit att_unit(const LoopParams& p, int u, int rank) {
  AttUnit a;
  a.rt = u % p.n_row_tiles; u /= p.n_row_tiles;
  a.kvh = u % p.n_kv_heads; a.b = u / p.n_kv_heads;
  a.plen = p.plen[a.b];
  a.npb = (a.plen + attn::KEY_BLOCK - 1) / attn::KEY_BLOCK;
  a.nkb = a.npb + (p.n_tok + attn::KEY_BLOCK - 1) / attn::KEY_BLOCK;
  a.kb0 = rank * a.nkb / CS; a.kb1 = (rank + 1) * a.nkb / CS;
  a.tok0 = a.b * p.n_tok;
  return a;
}

// ---- role: weight producer (projections) and K/V loader (attention) ------------------------------
template <int DH>
__device__ void role_weights(const Ctx& c) {
  const LoopParams& p = *c.p;
  Misc* ms = c.ms;
  constexpr int KVB = attn::KEY_BLOCK * DH * 2;
  const int C = p.n_clusters;
  int wslot = 0; uint32_t wphase = 0;
  uint32_t kv_cnt = 0;
  int nreal = 0, nlv = 0;
  bool ok = true;
  const uint64_t pol = ptx::policy_evict_first();
  const int G = p.n_q_heads / p.n_kv_heads;
  (void)G;
  walk_levels(p, [&](const Lv& lv) {
    if (!ok || !participates(lv, c.cid, C)) return;
    ++nlv;
    if (lv.units == 0) return;
    for (int u = first_unit(lv, c.cid, C); u < lv.units && ok; u += C) {
      if (lv.type == LV_ATT) {
        // the attention buffers overlay the weight ring: every tile requested so far must have been consumed
        for (int j = 0; j < NSW && ok; ++j) {
          const int s = (wslot + j) % NSW;
          const uint32_t ph = (wslot + j >= NSW) ? (wphase ^ 1u) : wphase;
          if (!bwait<false>(c, &ms->wempty[s], ph ^ 1u)) ok = false;
        }
        if (ok && !wait_count(c, &ms->units_done, nreal)) ok = false;
        if (!ok) break;
        const AttUnit a = att_unit(p, u, c.rank);
        bool flag_seen = false;
        const int k_off = p.n_q_heads * DH, v_off = k_off + p.n_kv_heads * DH;
        for (int blk = a.kb0; blk < a.kb1 && ok; ++blk, ++kv_cnt) {
          const int st = kv_cnt & 1;
          const uint32_t par = (kv_cnt >> 1) & 1u;
          uint8_t* kd = c.pool + OFF_K + st * KVB;
          uint8_t* vd = c.pool + OFF_V + st * KVB;
          if (blk < a.npb) {
            const int plane_k = (lv.l * 2 + 0) * p.n_kv_heads + a.kvh, plane_v = (lv.l * 2 + 1) * p.n_kv_heads + a.kvh;
            if (!bwait(c, &ms->k_empty[st], par ^ 1u)) { ok = false; break; }
            ptx::mbar_arrive_expect_tx(&ms->k_full[st], KVB);
            for (int j = 0; j < DH / 64; ++j)
              ptx::tma_load_3d(kd + j * (attn::KEY_BLOCK * 128), &p.pk[a.b], j * 64, blk * attn::KEY_BLOCK, plane_k, &ms->k_full[st]);
            if (!bwait(c, &ms->v_empty[st], par ^ 1u)) { ok = false; break; }
            ptx::mbar_arrive_expect_tx(&ms->v_full[st], KVB);
            for (int j = 0; j < DH / 64; ++j)
              ptx::tma_load_3d(vd + j * (attn::KEY_BLOCK * 128), &p.pk[a.b], j * 64, blk * attn::KEY_BLOCK, plane_v, &ms->v_full[st]);
          } else {
            if (!flag_seen) {  // the suffix keys are this step's: wait for the level's flag (seen by the polling thread)
              // (this thread runs ahead of the levels: a count, not the level barrier's parity)
              if (!wait_count(c, &ms->level_seen, nlv)) { ok = false; break; }
              ptx::fence_proxy_async_all();
              flag_seen = true;
            }
            const int row = a.tok0 + (blk - a.npb) * attn::KEY_BLOCK;
            if (!bwait(c, &ms->k_empty[st], par ^ 1u)) { ok = false; break; }
            ptx::mbar_arrive_expect_tx(&ms->k_full[st], KVB);
            for (int j = 0; j < DH / 64; ++j)
              ptx::tma_load_2d(kd + j * (attn::KEY_BLOCK * 128), &p.kv2d, k_off + a.kvh * DH + j * 64, row, &ms->k_full[st]);
            if (!bwait(c, &ms->v_empty[st], par ^ 1u)) { ok = false; break; }
            ptx::mbar_arrive_expect_tx(&ms->v_full[st], KVB);
            for (int j = 0; j < DH / 64; ++j)
              ptx::tma_load_2d(vd + j * (attn::KEY_BLOCK * 128), &p.kv2d, v_off + a.kvh * DH + j * 64, row, &ms->v_full[st]);
          }
        }
        // no weight may land in these bytes before the unit is over
        if (ok && !wait_count(c, &ms->units_done, nreal + 1)) ok = false;
        ++nreal;
      } else {
        const int gi = level_gemm(lv.type);
        const GemmLv& g = p.g[gi];
        const GemmUnit gu = gemm_unit(g, u, c.rank);
        if (!gu.valid) continue;
        const CUtensorMap* mw = p.maps + (gi == G_W2 ? MAP_W2 : MAP_LAYER0 + lv.l * 4 + (gi - 1));
        const int nv = g.dual ? 2 : 1;
        for (int i = 0; i < g.kbn && ok; ++i) {
          for (int v = 0; v < nv; ++v) {
            if (!bwait<false>(c, &ms->wempty[wslot], wphase ^ 1u)) { ok = false; break; }
            ptx::mbar_arrive_expect_tx(&ms->wfull[wslot], W_SLOT);
            ptx::tma_load_2d_hint(c.pool + OFF_W + wslot * W_SLOT, mw, (gu.sl * g.kbn + i) * 64, gu.ft * 128 * nv + v * 128,
                                  &ms->wfull[wslot], pol);
            if (++wslot == NSW) { wslot = 0; wphase ^= 1u; }
          }
        }
        ++nreal;
      }
    }
  });
  if (!ok) fail(c);
}

// ---- role: flag poller, activation loader (projections), Q loader (attention) ---------------------
template <int DH>
__device__ void role_acts(const Ctx& c) {
  const LoopParams& p = *c.p;
  Misc* ms = c.ms;
  const int C = p.n_clusters;
  int aslot = 0; uint32_t aphase = 0;
  uint32_t q_cnt = 0;
  int nreal = 0, nlv = 0;
  bool ok = true;
  const int G = p.n_q_heads / p.n_kv_heads;
  walk_levels(p, [&](const Lv& lv) {
    if (!ok || !participates(lv, c.cid, C)) return;
    if (lv.dep >= 0 && !poll_counter(c, p.counters + lv.dep, lv.dep_target)) { ok = false; return; }
    ptx::fence_proxy_async_all();
    ms->level_seen = ++nlv;
    __threadfence_block();
    ptx::mbar_arrive(&ms->level_go);
    if (lv.units == 0) return;
    for (int u = first_unit(lv, c.cid, C); u < lv.units && ok; u += C) {
      if (lv.type == LV_ATT) {
        const AttUnit a = att_unit(p, u, c.rank);
        // the query tile overlays the activation ring (and the previous unit's merge buffer)
        for (int j = 0; j < NSA && ok; ++j) {
          const int s = (aslot + j) % NSA;
          const uint32_t ph = (aslot + j >= NSA) ? (aphase ^ 1u) : aphase;
          if (!bwait<false>(c, &ms->aempty[s], ph ^ 1u)) ok = false;
        }
        if (ok && nreal > 0 && !bwait<false>(c, &ms->unit_done, (uint32_t)(nreal - 1) & 1u)) ok = false;
        if (!ok) break;
        if (a.kb1 > a.kb0) {
          ptx::mbar_arrive_expect_tx(&ms->q_full, 128 * DH * 2);
          for (int j = 0; j < DH / 64; ++j)
            ptx::tma_load_3d(c.pool + OFF_Q + j * (128 * 128), &p.maps[MAP_Q3D], j * 64, a.kvh * G, a.tok0 + a.rt * (128 / G), &ms->q_full);
          ++q_cnt;
        }
        ++nreal;
      } else {
        const GemmLv& g = p.g[level_gemm(lv.type)];
        const GemmUnit gu = gemm_unit(g, u, c.rank);
        if (!gu.valid) continue;
        const CUtensorMap* ma = p.maps + g.map_a;
        for (int i = 0; i < g.kbn; ++i) {
          if (!bwait<false>(c, &ms->aempty[aslot], aphase ^ 1u)) { ok = false; break; }
          ptx::mbar_arrive_expect_tx(&ms->afull[aslot], A_SLOT);
          ptx::tma_load_2d(c.pool + OFF_A + aslot * A_SLOT, ma, (gu.sl * g.kbn + i) * 64, 0, &ms->afull[aslot]);
          if (++aslot == NSA) { aslot = 0; aphase ^= 1u; }
        }
        ++nreal;
      }
    }
  });
  (void)q_cnt;
  if (!ok) fail(c);
}

// ---- role: MMA issuer of the projections and of S = Q K^T -----------------------------------------
template <int DH>
__device__ void role_mma(const Ctx& c) {
  const LoopParams& p = *c.p;
  Misc* ms = c.ms;
  constexpr int KVB = attn::KEY_BLOCK * DH * 2;
  const int C = p.n_clusters;
  int wslot = 0, aslot = 0; uint32_t wphase = 0, aphase = 0;
  uint32_t kv_cnt = 0, q_cnt = 0;
  int nreal = 0;
  bool ok = true;
  const uint32_t idesc = ptx::idesc_bf16_f32(128, TOK);
  const uint64_t wdesc0 = ptx::smem_desc_sw128(ptx::smem_u32(c.pool + OFF_W)), adesc0 = ptx::smem_desc_sw128(ptx::smem_u32(c.pool + OFF_A));
  const uint32_t idesc_s = ptx::idesc_bf16_f32(128, attn::KEY_BLOCK);
  const uint32_t tm_s = c.tmem + 256;
  walk_levels(p, [&](const Lv& lv) {
    if (!ok || lv.units == 0) return;
    for (int u = first_unit(lv, c.cid, C); u < lv.units && ok; u += C) {
      if (lv.type == LV_ATT) {
        const AttUnit a = att_unit(p, u, c.rank);
        const int nb = a.kb1 - a.kb0;
        if (nreal > 0 && !bwait<false>(c, &ms->unit_done, (uint32_t)(nreal - 1) & 1u)) { ok = false; break; }
        if (nb > 0) {
          if (!bwait(c, &ms->q_full, q_cnt & 1u)) { ok = false; break; }
          ++q_cnt;
          for (int i = 0; i < nb; ++i, ++kv_cnt) {
            const int s = kv_cnt & 1;
            const uint32_t par = (kv_cnt >> 1) & 1u;
            if (!bwait(c, &ms->k_full[s], par) || !bwait(c, &ms->s_empty[s], par ^ 1u)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t qa = ptx::smem_u32(c.pool + OFF_Q), ka = ptx::smem_u32(c.pool + OFF_K + s * KVB);
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
              ptx::umma_f16(tm_s + s * attn::KEY_BLOCK, ptx::smem_desc_sw128(qa + (ks >> 2) * (128 * 128) + (ks & 3) * 32),
                            ptx::smem_desc_sw128(ka + (ks >> 2) * (attn::KEY_BLOCK * 128) + (ks & 3) * 32), idesc_s, ks > 0);
            ptx::umma_commit(&ms->s_full[s]);
            ptx::umma_commit(&ms->k_empty[s]);
          }
        }
        ++nreal;
      } else {
        const GemmLv& g = p.g[level_gemm(lv.type)];
        const GemmUnit gu = gemm_unit(g, u, c.rank);
        if (!gu.valid) continue;
        if (nreal > 0 && !bwait<false>(c, &ms->unit_done, (uint32_t)(nreal - 1) & 1u)) { ok = false; break; }
        ptx::tc_fence_after();
        const int nv = g.dual ? 2 : 1;
        unsigned long long* tr = p.trace ? p.trace + ((size_t)lv.seq * c.n_cta + c.cta) * 8 : nullptr;
        for (int i = 0; i < g.kbn && ok; ++i) {
          if (!bwait(c, &ms->afull[aslot], aphase)) { ok = false; break; }
          if (tr && i == 0) tr[6] = ptx::globaltimer_ns();
          // descriptors differ from the first slot's only in the start-address field (16-byte units)
          const uint64_t ad = adesc0 + (uint64_t)(aslot * (A_SLOT >> 4));
          for (int v = 0; v < nv; ++v) {
            if (!bwait(c, &ms->wfull[wslot], wphase)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint64_t wd = wdesc0 + (uint64_t)(wslot * (W_SLOT >> 4));
            const uint32_t d = c.tmem + (uint32_t)(v * TOK);
            ptx::umma_f16(d, wd, ad, idesc, i > 0 ? 1u : 0u);
            ptx::umma_f16(d, wd + 2, ad + 2, idesc, 1u);
            ptx::umma_f16(d, wd + 4, ad + 4, idesc, 1u);
            ptx::umma_f16(d, wd + 6, ad + 6, idesc, 1u);
            ptx::umma_commit(&ms->wempty[wslot]);
            if (++wslot == NSW) { wslot = 0; wphase ^= 1u; }
          }
          ptx::umma_commit(&ms->aempty[aslot]);
          if (++aslot == NSA) { aslot = 0; aphase ^= 1u; }
        }
        if (ok) ptx::umma_commit(&ms->acc_full);
        if (tr) tr[7] = ptx::globaltimer_ns();
        ++nreal;
      }
    }
  });
  if (!ok) fail(c);
}

// ---- role: issuer of O += P V ------------------------------------------------------------------------
template <int DH>
__device__ void role_pv(const Ctx& c) {
  const LoopParams& p = *c.p;
  Misc* ms = c.ms;
  constexpr int KVB = attn::KEY_BLOCK * DH * 2;
  constexpr int P_BYTES = 128 * attn::KEY_BLOCK * 2;
  const int C = p.n_clusters;
  uint32_t kv_cnt = 0;
  int nreal = 0;
  bool ok = true;
  const uint32_t idesc_o = ptx::idesc_bf16_f32(128, DH) | (1u << 16);  // B (= V) is MN-major
  walk_levels(p, [&](const Lv& lv) {
    if (!ok || lv.units == 0) return;
    for (int u = first_unit(lv, c.cid, C); u < lv.units && ok; u += C) {
      if (lv.type != LV_ATT) {
        if (gemm_unit(p.g[level_gemm(lv.type)], u, c.rank).valid) ++nreal;
        continue;
      }
      const AttUnit a = att_unit(p, u, c.rank);
      const int nb = a.kb1 - a.kb0;
      if (nreal > 0 && !bwait<false>(c, &ms->unit_done, (uint32_t)(nreal - 1) & 1u)) { ok = false; break; }
      for (int i = 0; i < nb; ++i, ++kv_cnt) {
        const int s = kv_cnt & 1;
        const uint32_t par = (kv_cnt >> 1) & 1u;
        if (!bwait(c, &ms->p_full[s], par) || !bwait(c, &ms->v_full[s], par)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t pa = ptx::smem_u32(c.pool + OFF_P + s * P_BYTES), va = ptx::smem_u32(c.pool + OFF_V + s * KVB);
#pragma unroll
        for (int k4 = 0; k4 < attn::KEY_BLOCK / 16; ++k4)
          ptx::umma_f16(c.tmem, ptx::smem_desc_sw128(pa + k4 * 32), ptx::smem_desc_mn_sw128(va + k4 * 16 * 128, attn::KEY_BLOCK * 128),
                        idesc_o, (i > 0 || k4 > 0) ? 1u : 0u);
        ptx::umma_commit(&ms->pv_done[s]);
        ptx::umma_commit(&ms->v_empty[s]);
      }
      ++nreal;
    }
  });
  if (!ok) fail(c);
}

// ---- epilogue warps: helpers --------------------------------------------------------------------------
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t swz(int r, int ch) { return (uint32_t)(r * 128 + ((ch ^ (r & 7)) << 4)); }

// One level's flag: all of this block's stores of the level are ordered before the increment.
__device__ __forceinline__ bool publish(const Ctx& c, int type, int et, bool first_piece, int& nsync) {
  if (!epi_sync(c, nsync)) return false;
  if (et == 0) {
    if (c.p->debug_skip_level == type && first_piece) return true;  // test aid: a completion signal that never comes
    ptx::red_release_gpu_add(c.p->counters + type, 1u);
  }
  return true;
}

// Level spread over all blocks: ez = bf16(silu(x Wf + bf + c_k)) for the action rows (first layer of the action-time
// MLP with the action projection folded in) and the state token's rows of h / hb / sums of squares.
__device__ void level_embed_in(const Ctx& c, const Lv& lv, int et) {
  const LoopParams& p = *c.p;
  const int ncc = p.D / 128, nrb = (p.Ma + 3) / 4;
  const int main_items = nrb * ncc, items = main_items + p.B * ncc;
  const float* cvec = p.ctime + (int64_t)lv.k * p.D;
  for (int it = c.cta; it < items; it += c.n_cta) {
    if (it < main_items) {
      const int rb = it / ncc, cc = it - rb * ncc;
      const int col = cc * 128 + et, m0 = rb * 4;
      const float bias = p.bfold[col] + cvec[col];
      float acc[4] = {bias, bias, bias, bias};
      const float* wr = p.Wfold + (int64_t)col * p.A;
      // eight inputs per pass so that the loads of a pass are in flight together
      for (int j0 = 0; j0 < p.A; j0 += 8) {
        float w[8], xv[4][8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int jj = min(j0 + j, p.A - 1);
          w[j] = j0 + j < p.A ? __ldg(wr + jj) : 0.f;
#pragma unroll
          for (int r = 0; r < 4; ++r) xv[r][j] = __ldcg(p.x + (int64_t)min(m0 + r, p.Ma - 1) * p.A + jj);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int r = 0; r < 4; ++r) acc[r] = fmaf(xv[r][j], w[j], acc[r]);
      }
#pragma unroll
      for (int r = 0; r < 4; ++r)
        if (m0 + r < p.Ma) p.ez[(int64_t)(m0 + r) * p.D + col] = __float2bfloat16_rn(silu_f(acc[r]));
    } else {
      const int i2 = it - main_items, b = i2 / ncc, cc = i2 - b * ncc;
      const int col = cc * 128 + et;
      const int64_t row = (int64_t)b * p.n_tok;
      p.h[row * p.D + col] = p.hs[(int64_t)b * p.D + col];
      p.hb[row * p.D + col] = p.hsb[(int64_t)b * p.D + col];
      if (cc == 0 && et < p.n_dtiles) p.ssq[(int64_t)et * p.ssq_ld + row] = et == 0 ? p.ssq_state[b] : 0.f;
    }
  }
}

// Level spread over all blocks: v = rmsnorm(h_row) Wout' + bout for the action rows, x += dt v (and the call's output
// after the last step).  An item is (action row, one of 8 groups of outputs); each of the 4 warps takes outputs.
__device__ bool level_final(const Ctx& c, const Lv& lv, int et, int& nsync) {
  const LoopParams& p = *c.p;
  const int lane = et & 31, ew = et >> 5;
  const int parts = p.A >= 8 ? 8 : 1, per_part = (p.A + parts - 1) / parts;
  float4* srow = reinterpret_cast<float4*>(c.pool + OFF_A);  // (free: activations only arrive after a later level's flag)
  float* red = c.ms->red;
  const bool last = lv.k == p.K - 1;
  for (int it = c.cta; it < p.Ma * parts; it += c.n_cta) {
    const int m = it / parts, part = it - m * parts;
    const int j_end = min(p.A, (part + 1) * per_part);
    const float4* row = reinterpret_cast<const float4*>(p.h + ((int64_t)m + m / p.horizon + 1) * p.D);
    float ss = 0.f;
    if (!epi_sync(c, nsync)) return false;
#pragma unroll 2
    for (int d = et; d < p.D / 4; d += 128) {
      const float4 v = __ldcg(row + d);
      srow[d] = v;
      ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) red[ew] = ss;
    if (!epi_sync(c, nsync)) return false;
    const float tot = ((red[0] + red[1]) + red[2]) + red[3];
    const float rstd = 1.0f / sqrtf(tot / (float)p.D + p.eps);
    for (int j = part * per_part + ew; j < j_end; j += 4) {
      const float4* wr = reinterpret_cast<const float4*>(p.Wout + (int64_t)j * p.D);
      float a = 0.f;
#pragma unroll 4
      for (int d = lane; d < p.D / 4; d += 32) {
        const float4 w4 = __ldg(wr + d), v = srow[d];
        a = fmaf(v.x, w4.x, a); a = fmaf(v.y, w4.y, a); a = fmaf(v.z, w4.z, a); a = fmaf(v.w, w4.w, a);
      }
      for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      if (lane == 0) {
        const float xn = __ldcg(p.x + (int64_t)m * p.A + j) + p.dt * (a * rstd + p.bout[j]);
        p.x[(int64_t)m * p.A + j] = xn;
        if (last) p.out[(int64_t)m * p.A + j] = xn;
      }
    }
  }
  return true;
}


// Signal "this warp's partial sums are in the scratch" to every block of the cluster (one arrival per warp and
// block on each xfull barrier): a cluster-scope fence after the warp's stores, then relaxed remote arrivals.
__device__ __forceinline__ void signal_partials(const Ctx& c) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) {
    asm volatile("fence.acq_rel.cluster;" ::: "memory");
    const uint32_t bar = ptx::smem_u32(&c.ms->xfull);
    for (int r = 0; r < CS; ++r) ptx::mbar_arrive_remote_relaxed(ptx::mapa_shared(bar, r));
  }
}
// Wait for all partial sums of the cluster's current unit (acquire at cluster scope once the phase is complete).
__device__ __forceinline__ bool wait_partials(const Ctx& c, uint32_t parity) {
  if (!warp_wait(c, &c.ms->xfull, parity)) return false;
  asm volatile("fence.acq_rel.cluster;" ::: "memory");
  return true;
}
__device__ __forceinline__ void release_scratch(const Ctx& c, int et) {
  if (et == 0) {
    const uint32_t bar = ptx::smem_u32(&c.ms->xfree);
    for (int r = 0; r < CS; ++r) ptx::mbar_arrive_remote_relaxed(ptx::mapa_shared(bar, r));
  }
}
__device__ __forceinline__ float4 f4add(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }

// Second half of a projection unit's epilogue.  This block owns tpo = 64 / ks tokens of the tile; warp w takes the
// tokens my_tok0 + w, + 4, ... (tpw = tpo / 4 of them), lane q the features 4q .. 4q + 3.  Every value is the sum of
// the ks partials in slice order; tpw * ks = 16 loads per lane (and gate/up part) are in flight together.
template <int NV>
__device__ __forceinline__ void finalize_owned(const Ctx& c, const GemmLv& g, const GemmUnit& gu, int n_tok_valid, int lane, int ew,
                                               const float4 (&old4)[8], float rs_lane) {
  const LoopParams& p = *c.p;
  const int tpo = TOK / g.ks, tpw = tpo >> 2, my_tok0 = gu.sl * tpo;
  const float* xs = reinterpret_cast<const float*>(p.xscratch + (size_t)c.cid * XS_CLUSTER_BYTES);
  const int ksh = g.ks == 8 ? 3 : g.ks == 4 ? 2 : 1;
  float4 buf[16 * NV];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int t = i >> ksh, sl = i & (g.ks - 1);  // token slot, source slice
    const int tok = my_tok0 + ew + 4 * t;
    const int src = gu.grp * g.ks + sl;
#pragma unroll
    for (int vv = 0; vv < NV; ++vv)
      buf[i * NV + vv] = tok < n_tok_valid ? __ldcg(reinterpret_cast<const float4*>(xs + ((size_t)((src * 2 + vv) * TOK + tok)) * 128) + lane)
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float4 sum[8 * NV];
  if (g.ks == 8) {
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
      for (int vv = 0; vv < NV; ++vv) {
        float4 a = buf[(t * 8) * NV + vv];
#pragma unroll
        for (int q = 1; q < 8; ++q) a = f4add(a, buf[(t * 8 + q) * NV + vv]);
        sum[t * NV + vv] = a;
      }
  } else if (g.ks == 4) {
#pragma unroll
    for (int t = 0; t < 4; ++t)
#pragma unroll
      for (int vv = 0; vv < NV; ++vv) {
        float4 a = buf[(t * 4) * NV + vv];
#pragma unroll
        for (int q = 1; q < 4; ++q) a = f4add(a, buf[(t * 4 + q) * NV + vv]);
        sum[t * NV + vv] = a;
      }
  } else {
#pragma unroll
    for (int t = 0; t < 8; ++t)
#pragma unroll
      for (int vv = 0; vv < NV; ++vv) sum[t * NV + vv] = f4add(buf[(t * 2) * NV + vv], buf[(t * 2 + 1) * NV + vv]);
  }
  const int col = gu.ft * 128 + 4 * lane;
  float4 bias4 = make_float4(0.f, 0.f, 0.f, 0.f);
  if (g.epi == LEPI_EMBED) bias4 = *reinterpret_cast<const float4*>(p.b2 + col);
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    if (t < tpw) {
      const int tok = my_tok0 + ew + 4 * t;
      const bool tv = tok < n_tok_valid;
      const float4 v = sum[t * NV];
      if (g.epi == LEPI_STORE) {
        const float r = __shfl_sync(0xffffffffu, rs_lane, t);
        if (tv) *reinterpret_cast<uint2*>(p.qkv + (int64_t)tok * g.ldo + col) = make_uint2(attn::pack_bf16(v.x * r, v.y * r), attn::pack_bf16(v.z * r, v.w * r));
      } else if (g.epi == LEPI_GEGLU) {
        const float r = __shfl_sync(0xffffffffu, rs_lane, t);
        const float4 u = sum[t * NV + (NV - 1)];
        if (tv)
          *reinterpret_cast<uint2*>(p.mlp + (int64_t)tok * g.ldo + col) =
              make_uint2(attn::pack_bf16(tc::gelu_tanh_fast(v.x * r) * (u.x * r), tc::gelu_tanh_fast(v.y * r) * (u.y * r)),
                         attn::pack_bf16(tc::gelu_tanh_fast(v.z * r) * (u.z * r), tc::gelu_tanh_fast(v.w * r) * (u.w * r)));
      } else {
        float4 hv;
        int64_t rowi;
        if (g.epi == LEPI_RESID) { hv = f4add(old4[t], v); rowi = tok; }
        else { hv = f4add(v, bias4); rowi = tok + tok / p.horizon + 1; }
        float sq = (hv.x * hv.x + hv.y * hv.y) + (hv.z * hv.z + hv.w * hv.w);
        for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        if (tv) {
          *reinterpret_cast<float4*>(p.h + rowi * p.D + col) = hv;
          *reinterpret_cast<uint2*>(p.hb + rowi * p.D + col) = make_uint2(attn::pack_bf16(hv.x, hv.y), attn::pack_bf16(hv.z, hv.w));
          if (lane == 0) p.ssq[(int64_t)gu.ft * p.ssq_ld + rowi] = sq;
        }
      }
    }
  }
}

// ---- role: epilogue of the projections, softmax of the attention, element-wise levels ---------------
template <int DH>
__device__ void role_epilogue(const Ctx& c) {
  const LoopParams& p = *c.p;
  Misc* ms = c.ms;
  constexpr int KVB = attn::KEY_BLOCK * DH * 2;
  (void)KVB;
  constexpr int P_BYTES = 128 * attn::KEY_BLOCK * 2;
  const int C = p.n_clusters;
  const int et = threadIdx.x - 128, lane = et & 31, ew = et >> 5;  // ew = TMEM lane quarter (warp id % 4)
  const uint32_t lane_addr = (uint32_t)(ew * 32) << 16;
  const int G = p.n_q_heads / p.n_kv_heads, R = p.n_tok * G;
  const uint32_t tm_s = c.tmem + 256;
  int nlv = 0, nreal = 0, ngemm = 0, nx = 0, nsync = 0;
  uint32_t kv_cnt = 0;
  bool ok = true;
  walk_levels(p, [&](const Lv& lv) {
    if (!ok || !participates(lv, c.cid, C)) return;
    if (!warp_wait(c, &ms->level_go, (uint32_t)nlv & 1u)) { ok = false; return; }
    ++nlv;
    unsigned long long* tr = (p.trace && et == 0) ? p.trace + ((size_t)lv.seq * c.n_cta + c.cta) * 8 : nullptr;
    if (tr) tr[0] = ptx::globaltimer_ns();
    if (lv.units == 0) {
      if (tr) { tr[1] = (unsigned long long)clock64(); tr[2] = ptx::globaltimer_ns(); }
      if (lv.type == LV_EMBED_IN) level_embed_in(c, lv, et);
      else if (!level_final(c, lv, et, nsync)) { ok = false; return; }
      if (!publish(c, lv.type, et, lv.k == 0 && c.cta == 0, nsync)) { ok = false; return; }
      if (tr) { tr[3] = (unsigned long long)clock64(); tr[5] = ptx::globaltimer_ns(); }
      return;
    }
    bool first_unit_of_level = true;
    for (int u = first_unit(lv, c.cid, C); u < lv.units && ok; u += C, first_unit_of_level = false) {
      const bool first_piece = lv.k == 0 && lv.l == 0 && u == 0 && c.rank == 0;  // (the piece the test aid withholds)
      if (lv.type == LV_ATT) {
        // ================================ attention unit ================================
        const AttUnit a = att_unit(p, u, c.rank);
        const int nb = a.kb1 - a.kb0;
        const int row = et;
        float m_ref = -INFINITY, l = 0.f;
        for (int i = 0; i < nb && ok; ++i) {
          const uint32_t n = kv_cnt + i;
          const int s = n & 1;
          const uint32_t par = (n >> 1) & 1u;
          if (!warp_wait(c, &ms->s_full[s], par)) { ok = false; break; }
          ptx::tc_fence_after();
          float sc[64];
          ptx::tmem_ld_32x32(tm_s + s * attn::KEY_BLOCK + lane_addr, sc);
          ptx::tmem_ld_32x32(tm_s + s * attn::KEY_BLOCK + 32 + lane_addr, sc + 32);
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ms->s_empty[s]);
          // keys of this block that exist: prefix blocks end at prefix_len, suffix blocks at the token count
          const int blk = a.kb0 + i;
          const int nvalid = blk < a.npb ? min(attn::KEY_BLOCK, a.plen - blk * attn::KEY_BLOCK)
                                         : min(attn::KEY_BLOCK, p.n_tok - (blk - a.npb) * attn::KEY_BLOCK);
          if (nvalid < attn::KEY_BLOCK) {
#pragma unroll
            for (int j = 0; j < 64; ++j)
              if (j >= nvalid) sc[j] = -INFINITY;
          }
          // variant: the state token's rows (rows 0 .. G-1 of row tile 0) see, of the suffix, only the state token's key
          if (p.state_mask && a.rt * 128 + row < G && blk >= a.npb) {
            const int first = (blk - a.npb) * attn::KEY_BLOCK;
#pragma unroll
            for (int j = 0; j < 64; ++j)
              if (first + j > 0) sc[j] = -INFINITY;
          }
          float mx[4] = {sc[0], sc[1], sc[2], sc[3]};
#pragma unroll
          for (int j = 4; j < 64; j += 4) {
            mx[0] = fmaxf(mx[0], sc[j]); mx[1] = fmaxf(mx[1], sc[j + 1]);
            mx[2] = fmaxf(mx[2], sc[j + 2]); mx[3] = fmaxf(mx[3], sc[j + 3]);
          }
          const float mb = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * p.scale_log2;
          float corr = 1.f;
          const bool grow = mb > m_ref + 8.f;
          if (grow) {
            corr = exp2f(m_ref - mb);
            m_ref = mb;
            l *= corr;
          }
          if (i > 0 && __any_sync(0xffffffffu, grow)) {
            const uint32_t q = n - 1;
            if (!warp_wait(c, &ms->pv_done[q & 1], (q >> 1) & 1u)) { ok = false; break; }
            ptx::tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < DH; c0 += 32) {
              float o[32];
              ptx::tmem_ld_32x32(c.tmem + c0 + lane_addr, o);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] *= corr;
              ptx::tmem_st_32x32(c.tmem + c0 + lane_addr, o);
            }
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
          }
          if (i >= 2) {
            const uint32_t q = n - 2;
            if (!warp_wait(c, &ms->pv_done[q & 1], (q >> 1) & 1u)) { ok = false; break; }
          }
          uint8_t* sPn = c.pool + OFF_P + s * P_BYTES;
          const float m_sub = m_ref == -INFINITY ? 0.f : m_ref;  // (all keys of the range masked for this row: exp2(-inf) = 0)
          float rs4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float p0 = ex2f(fmaf(sc[ch * 8 + 2 * q], p.scale_log2, -m_sub)), p1 = ex2f(fmaf(sc[ch * 8 + 2 * q + 1], p.scale_log2, -m_sub));
              rs4[q] += p0 + p1;
              w[q] = attn::pack_bf16(p0, p1);
            }
            *reinterpret_cast<uint4*>(sPn + swz(row, ch)) = make_uint4(w[0], w[1], w[2], w[3]);
          }
          l += (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
          ptx::fence_proxy_async();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ms->p_full[s]);
        }
        if (!ok) break;
        if (nb > 0) {
          const uint32_t q = kv_cnt + nb - 1;
          if (!warp_wait(c, &ms->pv_done[q & 1], (q >> 1) & 1u)) { ok = false; break; }
          ptx::tc_fence_after();
        }
        kv_cnt += nb;
        if (tr && first_unit_of_level) tr[1] = ptx::globaltimer_ns();
        // ---- merge of the 8 key ranges inside the cluster, through the scratch in global memory ----
        if (nx > 0 && !warp_wait(c, &ms->xfree, (uint32_t)(nx - 1) & 1u)) { ok = false; break; }
        {
          uint8_t* xs = p.xscratch + (size_t)c.cid * XS_CLUSTER_BYTES;
          uint4* dst = reinterpret_cast<uint4*>(xs + (size_t)c.rank * XS_BLOCK_BYTES + (size_t)row * (DH * 2));
          reinterpret_cast<float2*>(xs + XS_ML_OFF)[c.rank * 128 + row] = make_float2(m_ref, l);
#pragma unroll 1
          for (int c0 = 0; c0 < DH; c0 += 32) {
            float o[32];
            if (nb > 0) {
              ptx::tmem_ld_32x32(c.tmem + c0 + lane_addr, o);
              ptx::tmem_ld_wait();
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] = 0.f;
            }
#pragma unroll
            for (int j = 0; j < 32; j += 8)
              dst[(c0 + j) >> 3] = make_uint4(attn::pack_bf16(o[j], o[j + 1]), attn::pack_bf16(o[j + 2], o[j + 3]),
                                              attn::pack_bf16(o[j + 4], o[j + 5]), attn::pack_bf16(o[j + 6], o[j + 7]));
          }
          ptx::tc_fence_before();
        }
        signal_partials(c);
        if (!wait_partials(c, (uint32_t)nx & 1u)) { ok = false; break; }
        {
          // thread = (owned row, 1/8 of the channels): weights of the 8 ranges in fixed order
          constexpr int CPT = DH / 8;  // channels per thread
          const int rl = et >> 3, part = et & 7;
          const int rrow = c.rank * 16 + rl;  // row of the tile owned by this block
          const uint8_t* xs = p.xscratch + (size_t)c.cid * XS_CLUSTER_BYTES;
          float mm[CS], ll[CS];
          float M = -INFINITY;
#pragma unroll
          for (int s = 0; s < CS; ++s) {
            const float2 v = __ldcg(reinterpret_cast<const float2*>(xs + XS_ML_OFF) + s * 128 + rrow);
            mm[s] = v.x; ll[s] = v.y; M = fmaxf(M, v.x);
          }
          float L = 0.f;
#pragma unroll
          for (int s = 0; s < CS; ++s) { mm[s] = mm[s] == -INFINITY ? 0.f : exp2f(mm[s] - M); L += ll[s] * mm[s]; }
          const float inv = 1.0f / L;
          float acc[CPT];
#pragma unroll
          for (int e = 0; e < CPT; ++e) acc[e] = 0.f;
#pragma unroll
          for (int s0 = 0; s0 < CS; s0 += 4) {
            uint4 raw[4][CPT / 8];
#pragma unroll
            for (int s = 0; s < 4; ++s)
#pragma unroll
              for (int q = 0; q < CPT / 8; ++q)
                raw[s][q] = __ldcg(reinterpret_cast<const uint4*>(xs + (size_t)(s0 + s) * XS_BLOCK_BYTES + (size_t)rrow * (DH * 2) + part * CPT * 2) + q);
#pragma unroll
            for (int s = 0; s < 4; ++s)
#pragma unroll
              for (int q = 0; q < CPT / 8; ++q) {
                const uint32_t w[4] = {raw[s][q].x, raw[s][q].y, raw[s][q].z, raw[s][q].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  acc[q * 8 + 2 * k] = fmaf(__uint_as_float(w[k] << 16), mm[s0 + s], acc[q * 8 + 2 * k]);
                  acc[q * 8 + 2 * k + 1] = fmaf(__uint_as_float(w[k] & 0xffff0000u), mm[s0 + s], acc[q * 8 + 2 * k + 1]);
                }
              }
          }
          const int gr = a.rt * 128 + rrow;
          if (gr < R) {
            const int tok = gr / G, hq = a.kvh * G + (gr - tok * G);
            uint4* dstg = reinterpret_cast<uint4*>(p.att + (int64_t)(a.tok0 + tok) * (p.n_q_heads * DH) + hq * DH + part * CPT);
#pragma unroll
            for (int q = 0; q < CPT / 8; ++q)
              dstg[q] = make_uint4(attn::pack_bf16(acc[q * 8] * inv, acc[q * 8 + 1] * inv), attn::pack_bf16(acc[q * 8 + 2] * inv, acc[q * 8 + 3] * inv),
                                   attn::pack_bf16(acc[q * 8 + 4] * inv, acc[q * 8 + 5] * inv), attn::pack_bf16(acc[q * 8 + 6] * inv, acc[q * 8 + 7] * inv));
          }
        }
        ++nx;
        if (!publish(c, LV_ATT, et, first_piece, nsync)) { ok = false; break; }
        release_scratch(c, et);
        if (et == 0) { __threadfence_block(); ms->units_done = nreal + 1; }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ms->unit_done);
        ++nreal;
      } else {
        // ================================ projection unit ================================
        const int gi = level_gemm(lv.type);
        const GemmLv& g = p.g[gi];
        const GemmUnit gu = gemm_unit(g, u, c.rank);
        if (!gu.valid) {  // this block has no tile in the unit: it only keeps the counts going
          if (nx > 0 && !warp_wait(c, &ms->xfree, (uint32_t)(nx - 1) & 1u)) { ok = false; break; }
          signal_partials(c);
          release_scratch(c, et);
          if (!publish(c, lv.type, et, first_piece, nsync)) { ok = false; break; }
          ++nx;
          continue;
        }
        const int nv = g.dual ? 2 : 1;
        const int tpo = TOK / g.ks, tpw = tpo >> 2;  // tokens finalised by this block / by each of its warps
        const int my_tok0 = gu.sl * tpo;
        const int n_tok_valid = g.epi == LEPI_EMBED ? p.Ma : p.M;
        // what does not depend on the accumulator: 1/rms of this warp's tokens (lane t: token slot t), old residuals
        float rs_lane = 1.f;
        if ((g.epi == LEPI_STORE || g.epi == LEPI_GEGLU) && lane < tpw) {
          const int tok = my_tok0 + ew + 4 * lane;
          if (tok < n_tok_valid) {
            float tot = 0.f;
            for (int i = 0; i < p.n_dtiles; ++i) tot += __ldcg(p.ssq + (int64_t)i * p.ssq_ld + tok);
            rs_lane = 1.0f / sqrtf(tot / (float)p.D + p.eps);
          }
        }
        float4 old4[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const int tok = my_tok0 + ew + 4 * t;
          old4[t] = (g.epi == LEPI_RESID && t < tpw && tok < n_tok_valid)
                        ? __ldcg(reinterpret_cast<const float4*>(p.h + (int64_t)tok * p.D + gu.ft * 128) + lane)
                        : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (!warp_wait(c, &ms->acc_full, (uint32_t)ngemm & 1u)) { ok = false; break; }
        ptx::tc_fence_after();
        if (tr && first_unit_of_level) tr[1] = ptx::globaltimer_ns();
        if (nx > 0 && !warp_wait(c, &ms->xfree, (uint32_t)(nx - 1) & 1u)) { ok = false; break; }
        // partial sums -> scratch[this block][gate | up][token][feature]; thread = feature (TMEM lane)
        {
          float* xs = reinterpret_cast<float*>(p.xscratch + (size_t)c.cid * XS_CLUSTER_BYTES) + (size_t)c.rank * (2 * TOK * 128) + et;
#pragma unroll 1
          for (int vv = 0; vv < nv; ++vv) {
#pragma unroll 1
            for (int c0 = 0; c0 < TOK; c0 += 32) {
              float v[32];
              ptx::tmem_ld_32x32(c.tmem + (uint32_t)(vv * TOK + c0) + lane_addr, v);
              ptx::tmem_ld_wait();
              float* dst = xs + (size_t)(vv * TOK + c0) * 128;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (c0 + j < n_tok_valid) dst[j * 128] = v[j];
            }
          }
        }
        ptx::tc_fence_before();
        signal_partials(c);
        if (tr && first_unit_of_level) tr[2] = ptx::globaltimer_ns();
        if (!wait_partials(c, (uint32_t)nx & 1u)) { ok = false; break; }
        if (tr && first_unit_of_level) tr[3] = ptx::globaltimer_ns();
        if (nv == 2) finalize_owned<2>(c, g, gu, n_tok_valid, lane, ew, old4, rs_lane);
        else finalize_owned<1>(c, g, gu, n_tok_valid, lane, ew, old4, rs_lane);
        if (tr && first_unit_of_level) tr[4] = ptx::globaltimer_ns();
        if (!publish(c, lv.type, et, first_piece, nsync)) { ok = false; break; }
        release_scratch(c, et);
        if (et == 0) { __threadfence_block(); ms->units_done = nreal + 1; }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ms->unit_done);
        ++ngemm; ++nx; ++nreal;
      }
    }
    if (tr) tr[5] = ptx::globaltimer_ns();
  });
  if (!ok && lane == 0) fail(c);
}

// ---- the kernel -----------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(THREADS, 1) adit_loop_kernel(const __grid_constant__ LoopParams p) {
  extern __shared__ uint8_t smem_raw[];
  Misc* ms = reinterpret_cast<Misc*>(smem_raw + POOL);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool aligned = (ptx::smem_u32(smem_raw) & 1023u) == 0;  // the swizzled tiles need 1024-byte alignment
  if (threadIdx.x == 0) {
    for (int i = 0; i < NSW; ++i) { ptx::mbar_init(&ms->wfull[i], 1); ptx::mbar_init(&ms->wempty[i], 1); }
    for (int i = 0; i < NSA; ++i) { ptx::mbar_init(&ms->afull[i], 1); ptx::mbar_init(&ms->aempty[i], 1); }
    ptx::mbar_init(&ms->acc_full, 1);
    ptx::mbar_init(&ms->unit_done, 4);
    ptx::mbar_init(&ms->level_go, 1);
    ptx::mbar_init(&ms->xfull, CS * 4);
    ptx::mbar_init(&ms->xfree, CS);
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&ms->k_full[s], 1); ptx::mbar_init(&ms->k_empty[s], 1);
      ptx::mbar_init(&ms->v_full[s], 1); ptx::mbar_init(&ms->v_empty[s], 1);
      ptx::mbar_init(&ms->s_full[s], 1); ptx::mbar_init(&ms->s_empty[s], 4);
      ptx::mbar_init(&ms->p_full[s], 4); ptx::mbar_init(&ms->pv_done[s], 1);
    }
    ptx::mbar_init(&ms->q_full, 1);
    ptx::mbar_init(&ms->epi_bar, 4);
    ms->abort = 0;
    ms->level_seen = 0;
    ms->units_done = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 3) {
    ptx::tmem_alloc(&ms->tmem_base, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // every block of the cluster has initialised its barriers before any peer signals them
  ptx::cluster_arrive_release();
  ptx::cluster_wait_acquire();
  ptx::pdl_launch_dependents();
  // The call's set-up kernel (counters, x, state token) precedes this one in the stream; with programmatic dependent
  // launch this kernel's prologue above overlaps it, everything below comes after it.
  ptx::pdl_wait_prior_grids();

  Ctx c;
  c.p = &p; c.ms = ms; c.pool = smem_raw; c.tmem = ms->tmem_base;
  c.rank = (int)ptx::cluster_ctarank(); c.cid = blockIdx.x / CS; c.n_cta = gridDim.x; c.cta = blockIdx.x;
  if (!aligned) {
    if (threadIdx.x == 0) fail(c);
  } else if (warp == 0) {
    if (lane == 0) role_weights<DH>(c);
  } else if (warp == 1) {
    if (lane == 0) role_acts<DH>(c);
  } else if (warp == 2) {
    if (lane == 0) role_mma<DH>(c);
  } else if (warp == 3) {
    if (lane == 0) role_pv<DH>(c);
  } else {
    role_epilogue<DH>(c);
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (ms->abort) {
    // a wait gave up: let copies still in flight land before the block's memory is released
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) {}
    __syncthreads();
  }
  // no block leaves while a peer may still write into its shared memory
  ptx::cluster_arrive_release();
  ptx::cluster_wait_acquire();
  if (warp == 3) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(c.tmem, 512);
  }
}

// Before the loop kernel, once per call: zero the level counters and the abort word, x <- noise, and the state
// token hs[b] = state[b] Ws + bs with its bf16 copy and sum of squares (block b).
__global__ void __launch_bounds__(256) loop_setup_kernel(uint32_t* __restrict__ counters, const float* __restrict__ noise,
                                                         const float* __restrict__ state, float* __restrict__ x, int n_x,
                                                         const float* __restrict__ Ws, const float* __restrict__ bs,
                                                         float* __restrict__ hs, bf16* __restrict__ hsb,
                                                         float* __restrict__ ssq_state, int B, int S, int D) {
  __shared__ float red[8];
  ptx::pdl_launch_dependents();
  if (blockIdx.x == 0 && threadIdx.x < 2 * LV_COUNT) counters[threadIdx.x] = 0u;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_x; i += gridDim.x * blockDim.x) x[i] = noise[i];
  for (int b = blockIdx.x; b < B; b += gridDim.x) {
    float ss = 0.f;
    for (int n = threadIdx.x; n < D; n += blockDim.x) {
      float a = bs[n];
      for (int j = 0; j < S; ++j) a = fmaf(state[b * S + j], Ws[(int64_t)n * S + j], a);
      hs[(int64_t)b * D + n] = a;
      hsb[(int64_t)b * D + n] = __float2bfloat16_rn(a);
      ss = fmaf(a, a, ss);
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
      for (int w = 0; w < 8; ++w) t += red[w];
      ssq_state[b] = t;
    }
  }
}

}  // namespace loop
}  // namespace adit
