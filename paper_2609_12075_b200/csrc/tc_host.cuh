// Host side of the tensor-core projections: TMA descriptors, tile/split planning and launches.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "gemm_tc.cuh"
#include "gemm_pair.cuh"

namespace adit {
namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up at run time so that the library has no link-time
// dependency on libcuda (it must load on machines without a driver).
static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// Row-major bf16 matrix [rows, cols] (cols contiguous, cols % 64 == 0); boxes of box_rows x 64 elements with the
// 128-byte swizzle; rows outside the matrix read as zero.
static bool make_map_bf16(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)TILE_K, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Query rows of the attention kernel: bf16 [rows, ld] where each row starts with n_heads heads of dh channels.
// Seen as a 3-D tensor (channel, head, row); a box is 64 channels x `group` heads x 128 / group rows, i.e. 128
// (row, head) pairs in row-major order, 128 bytes each, 128-byte swizzle.
static bool make_map_q(CUtensorMap* m, const void* base, uint64_t rows, uint64_t ld, uint32_t dh, uint32_t n_heads,
                       uint32_t group) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || group == 0 || 128 % group || group > 128) return false;
  cuuint64_t gdim[3] = {dh, n_heads, rows};
  cuuint64_t gstride[2] = {(cuuint64_t)dh * 2, ld * 2};
  cuuint32_t box[3] = {64, group, 128 / group};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct GemmPlan {
  int tile_tok, n_ttiles, n_ftiles, splits, stages, kb_total, acc_bufs, issuers;
  uint32_t tmem_cols, ring_bytes;
  size_t smem_bytes;
  double est_us;  // the planner's estimate of the kernel's duration
  bool pair = false;  // the two-SM kernel (gemm_pair_kernel): tile_tok tokens x 256 features per pair of blocks
};

// Tile shape and k-split (= cluster size) depend on the problem size and the device's SM count only,
// never on the per-call SM budget, so that the summation order - and with it every output bit - is
// the same for any budget.
//
// The choice minimises an estimate of the kernel's duration built from figures measured on B200 with this
// kernel: a k-block costs the thread that issues the products about 0.37 us (0.49 us for a gate/up pair; with two
// issuing threads half of that, which is also what the tensor pipe itself then needs for narrow products: about 85
// cycles each whatever their width, since each fetches its 4 KB slab of weight rows from shared memory), more
// when shared memory (128 B per cycle for the incoming stage plus the operand reads of every product) or the
// block's intake (about 150 GB/s; the whole chip about 25 TB/s out of L2, weights about 6 TB/s out of HBM) is slower; the first operands arrive about 1 us after they were asked for; the epilogue
// costs about 0.5 us per 32 tokens (only the last tile's is exposed); and a k-split over a cluster adds
// parking the accumulator, the exchange through distributed shared memory (about 20 GB/s into each
// block), the rank-order sum and a cluster barrier.
static GemmPlan plan_gemm(int n_tok, int n_feat, int K, bool dual, int sm_count, bool allow_split, int force_splits = 0,
                          int force_ttiles = 0) {
  GemmPlan p;
  const int nv = dual ? 2 : 1;
  p.n_ftiles = (n_feat + TILE_F - 1) / TILE_F;
  p.kb_total = K / TILE_K;
  p.n_ttiles = (n_tok + 127) / 128; p.tile_tok = 128; p.splits = 1; p.acc_bufs = 2; p.issuers = 1;
  double best = 1e30;
  const double w_bytes = (double)p.n_ftiles * nv * TILE_F * K * 2;
  for (int nt = 1; nt <= 64; ++nt) {
    const int tile16 = (((n_tok + nt - 1) / nt) + 15) / 16 * 16;
    if (tile16 > 256) continue;
    if (nt > 1 && tile16 < 32) break;
    if (force_ttiles > 0 && nt != force_ttiles) continue;  // test aid
    for (int cs = 8; cs >= 1; cs >>= 1) {
      if (cs > 1 && !allow_split && force_splits <= 0) continue;
      if (force_splits > 0 && cs > force_splits) continue;
      if (cs > p.kb_total) continue;
      const int tile = cs > 1 ? (tile16 + 8 * cs - 1) / (8 * cs) * (8 * cs) : tile16;
      if (tile > 256 || nv * tile > 512) continue;
      const int64_t items = (int64_t)p.n_ftiles * nt, blocks = items * cs;
      if (cs > 1 && blocks > sm_count) continue;  // clusters of a k-split run as one wave
      const bool one_item = blocks <= sm_count;   // a single accumulator buffer serialises a block's tiles
      // Two issuers need two k-blocks each way and room for their own accumulators; they pay off while a
      // k-block's products are issued more slowly than they execute (narrow tiles).
      int issuers = 1, acc_bufs = 2 * nv * tile <= 512 ? 2 : 1;
      if (p.kb_total / cs >= 2 && nv * tile <= 208) {
        if (4 * nv * tile <= 512) { issuers = 2; acc_bufs = 2; }
        else if (2 * nv * tile <= 512 && one_item) { issuers = 2; acc_bufs = 1; }
      }
      if (acc_bufs == 1 && !one_item) continue;
      const size_t stage = (size_t)nv * TILE_F * TILE_K * 2 + (size_t)tile * TILE_K * 2;
      const size_t xbuf = cs > 1 ? 2 * (size_t)tile * TILE_F * 4 * nv : 0;
      if (xbuf + 2 * stage > (size_t)SMEM_BUDGET) continue;
      const int64_t active = blocks < sm_count ? blocks : sm_count;
      const int64_t waves = (blocks + sm_count - 1) / sm_count;
      const int kb_blk = (p.kb_total + cs - 1) / cs;
      // one k-block: the issuing thread needs about 0.25 us plus 0.03 us per product (4 or 8 of them); a block
      // takes in about 150 GB/s, the chip about 25 TB/s out of L2
      double t_kb = (0.25 + 0.03 * 4 * nv) / issuers;
      if (t_kb < 0.16) t_kb = 0.16;  // the producers need that long per stage
      // shared memory moves 128 bytes per cycle: the copy engine writes the stage, and every product reads its
      // 4 KB of weights and its 32 bytes per token again
      const double smem_traffic = (double)stage + 4.0 * nv * (4096.0 + 32.0 * tile);
      if (smem_traffic / 243e3 > t_kb) t_kb = smem_traffic / 243e3;
      if ((double)stage / 150e3 > t_kb) t_kb = (double)stage / 150e3;
      if ((double)active * (double)stage / 25e6 > t_kb) t_kb = (double)active * (double)stage / 25e6;
      double t_main = (double)waves * kb_blk * t_kb;
      if (w_bytes / 6e6 > t_main) t_main = w_bytes / 6e6;
      const int slice = tile / cs;
      double t_epi;
      if (cs == 1) {
        t_epi = 0.5 * ((tile + 31) / 32) * (dual ? 1.3 : 1.0);
      } else {
        t_epi = 0.25 * ((tile + 31) / 32) * nv + 0.6 + (double)cs * slice * nv * TILE_F * 4 / 20e3 +
                0.9 * ((slice + 31) / 32) * (dual ? 1.3 : 1.0) + 0.5;
      }
      const double t = 1.1 + t_main + t_epi;
      if (t < best - 1e-9) { best = t; p.n_ttiles = nt; p.tile_tok = tile; p.splits = cs; p.acc_bufs = acc_bufs; p.issuers = issuers; }
      if (force_splits > 0) break;  // test aid: take the largest admissible cluster for this tiling
    }
  }
  p.est_us = best;
  const int items = p.n_ftiles * p.n_ttiles;
  const size_t stage_bytes = (size_t)nv * TILE_F * TILE_K * 2 + (size_t)p.tile_tok * TILE_K * 2;
  const size_t xbuf_bytes = p.splits > 1 ? 2 * (size_t)p.tile_tok * TILE_F * 4 * nv : 0;  // send + receive
  p.stages = (int)((SMEM_BUDGET - xbuf_bytes) / stage_bytes);
  if (p.stages > MAX_STAGES) p.stages = MAX_STAGES;
  if ((int64_t)items * p.splits <= sm_count) {
    // one work item per block: a ring as deep as the item's k-blocks is enough, and the smaller
    // footprint lets the next kernel's blocks become resident (and prefetch) beside this one
    int kb_item = (p.kb_total + p.splits - 1) / p.splits;
    if (kb_item < 2) kb_item = 2;
    if (p.stages > kb_item) p.stages = kb_item;
  }
  // With two issuers the ring must have an even number of stages: every stage then belongs to one issuer, which
  // sees its fills in order.  (With an odd number a stage alternates between the issuers, and the one that runs
  // ahead could take the other's still pending fill for its own: a barrier's parity cannot tell them apart.)
  if (p.issuers == 2 && (p.stages & 1)) p.stages -= 1;
  p.ring_bytes = (uint32_t)(p.stages * stage_bytes);
  p.smem_bytes = (size_t)p.ring_bytes + xbuf_bytes + 1024;
  uint32_t need = (uint32_t)(p.acc_bufs * nv * p.issuers * p.tile_tok), cols = 32;
  while (cols < need) cols <<= 1;
  p.tmem_cols = cols;
  return p;
}

// Rows of the token operand's TMA box: a block of the two-SM kernel brings in half a tile.
static int token_box_rows(const GemmPlan& p) { return p.pair ? p.tile_tok / 2 : p.tile_tok; }

// Plan for the two-SM kernel: a pair of blocks owns tiles of 256 features x tile_tok tokens.  The tile width minimises
// rounds x (k-blocks x time per k-block + epilogue), in cycles: a k-block's products take 2 cycles per token (twice for
// a gate/up pair) at the tensor peak, shared memory (128 bytes per cycle) has to take in the stage and feed every
// product its weight rows and this block's half of the tokens, and the issuing thread needs about 45 cycles per
// product.  The model is coarse: it prefers the widest tiles, which is what measured best where this kernel is used.
// As for plan_gemm, nothing here depends on the call's SM budget.
static GemmPlan plan_gemm_pair(int n_tok, int n_feat, int K, bool dual, int sm_count) {
  GemmPlan p{};
  const int nv = dual ? 2 : 1;
  p.pair = true;
  p.n_ftiles = (n_feat + TILE_F - 1) / TILE_F;
  p.kb_total = K / TILE_K;
  p.splits = 1; p.issuers = 1;
  const int n_fpairs = (p.n_ftiles + 1) / 2, n_pairs = sm_count / 2 > 0 ? sm_count / 2 : 1;
  double best = 1e30;
  for (int nt = 1; nt <= 128; ++nt) {
    const int tile = (((n_tok + nt - 1) / nt) + 15) / 16 * 16;
    if (tile > 256) continue;
    if (nt > 1 && tile < 32) break;
    const int64_t rounds = ((int64_t)n_fpairs * nt + n_pairs - 1) / n_pairs;
    const int acc_bufs = 2 * nv * tile <= 512 ? 2 : 1;
    const double stage = nv * 16384.0 + tile * 64.0;
    double t_kb = 2.0 * nv * tile;                                          // products
    const double smem = (stage + nv * (16384.0 + tile * 64.0)) / 128.0;     // stage in + operand reads
    if (smem > t_kb) t_kb = smem;
    if (t_kb < 4.0 * nv * 45.0) t_kb = 4.0 * nv * 45.0;                     // issue rate of one thread
    const double t_epi = 12.0 * tile * (dual ? 1.3 : 1.0);                  // about 0.2 us per 32 tokens
    // with two accumulator buffers only the last tile's epilogue is exposed
    const double t = acc_bufs == 2 ? rounds * p.kb_total * t_kb + t_epi : rounds * (p.kb_total * t_kb + t_epi);
    if (t < best - 1e-9) { best = t; p.n_ttiles = nt; p.tile_tok = tile; p.acc_bufs = acc_bufs; }
  }
  p.est_us = 2.0 + best / 1900.0;  // (launch, set-up of the pair, first operands)
  const size_t stage_bytes = (size_t)nv * TILE_F * TILE_K * 2 + (size_t)(p.tile_tok / 2) * TILE_K * 2;
  p.stages = (int)(SMEM_BUDGET / stage_bytes);
  if (p.stages > MAX_STAGES) p.stages = MAX_STAGES;
  if ((int64_t)n_fpairs * p.n_ttiles <= n_pairs) {
    // one tile per pair: a ring as deep as the tile's k-blocks is enough (the smaller footprint lets the next
    // kernel's blocks become resident beside this one)
    int kb_item = p.kb_total < 2 ? 2 : p.kb_total;
    if (p.stages > kb_item) p.stages = kb_item;
  }
  p.ring_bytes = (uint32_t)(p.stages * stage_bytes);
  p.smem_bytes = (size_t)p.ring_bytes + 1024;
  uint32_t need = (uint32_t)(p.acc_bufs * nv * p.tile_tok), cols = 32;
  while (cols < need) cols <<= 1;
  p.tmem_cols = cols;
  return p;
}

// The plan a projection runs with.  Measured on B200 at 816 and 1632 tokens, the two-SM kernel beats the one-SM kernel
// (which has two issuing threads and finer tiles) only for the gate/up pair at the larger size - 33 against 36 us - and
// for large plain products (8192 x 2048 x 2048: 54 against 62 us); the other projections of these sizes are bound by
// fixed costs (set-up, first operands, the exposed epilogue of a single tile per block), where the pair's longer set-up
// loses.  So: gate/up pairs from PAIR_DUAL_MIN_TOKENS tokens on go to the two-SM kernel, everything else to the
// one-SM kernel with its k-split.  A function of the problem size and the device only.
constexpr int PAIR_DUAL_MIN_TOKENS = 1024;
static GemmPlan plan_projection(int n_tok, int n_feat, int K, bool dual, int sm_count, bool allow_pair) {
  if (allow_pair && dual && n_tok >= PAIR_DUAL_MIN_TOKENS && sm_count >= 2 && (K / TILE_K) >= 2)
    return plan_gemm_pair(n_tok, n_feat, K, dual, sm_count);
  return plan_gemm(n_tok, n_feat, K, dual, sm_count, true);
}

// One instantiation per (gate/up pair, epilogue) x chunk width x k-split x issuing threads x instrumentation: a
// launch then runs through (and has to fetch) only the code it needs.
template <bool D, int E, typename F>
static cudaError_t for_gemm_variant(int idx, F&& f) {
  switch (idx) {
#define ADIT_V(i, CW, SP, NI, IN) case i: return f(gemm_tc_kernel<D, E, CW, SP, NI, IN>);
    ADIT_V(0, 16, false, 1, false) ADIT_V(1, 32, false, 1, false) ADIT_V(2, 16, true, 1, false) ADIT_V(3, 32, true, 1, false)
    ADIT_V(4, 16, false, 2, false) ADIT_V(5, 32, false, 2, false) ADIT_V(6, 16, true, 2, false) ADIT_V(7, 32, true, 2, false)
    ADIT_V(8, 16, false, 1, true) ADIT_V(9, 32, false, 1, true) ADIT_V(10, 16, true, 1, true) ADIT_V(11, 32, true, 1, true)
    ADIT_V(12, 16, false, 2, true) ADIT_V(13, 32, false, 2, true) ADIT_V(14, 16, true, 2, true) ADIT_V(15, 32, true, 2, true)
#undef ADIT_V
    default: return cudaErrorInvalidValue;
  }
}
template <bool D, int E, typename F>
static cudaError_t for_pair_variant(int idx, F&& f) {
  switch (idx) {
    case 0: return f(gemm_pair_kernel<D, E, 16, false>);
    case 1: return f(gemm_pair_kernel<D, E, 32, false>);
    case 2: return f(gemm_pair_kernel<D, E, 16, true>);
    case 3: return f(gemm_pair_kernel<D, E, 32, true>);
    default: return cudaErrorInvalidValue;
  }
}
template <typename F>
static cudaError_t for_pair_kernel(bool dual, int epi, int idx, F&& f) {
  if (dual) return for_pair_variant<true, EPI_GEGLU>(idx, f);
  switch (epi) {
    case EPI_STORE: return for_pair_variant<false, EPI_STORE>(idx, f);
    case EPI_SILU_VEC: return for_pair_variant<false, EPI_SILU_VEC>(idx, f);
    case EPI_STORE_F32: return for_pair_variant<false, EPI_STORE_F32>(idx, f);
    case EPI_RESID_NORM: return for_pair_variant<false, EPI_RESID_NORM>(idx, f);
    case EPI_EMBED_NORM: return for_pair_variant<false, EPI_EMBED_NORM>(idx, f);
    default: return cudaErrorInvalidValue;
  }
}
template <typename F>
static cudaError_t for_gemm_kernel(bool dual, int epi, int idx, F&& f) {
  if (dual) return for_gemm_variant<true, EPI_GEGLU>(idx, f);
  switch (epi) {
    case EPI_STORE: return for_gemm_variant<false, EPI_STORE>(idx, f);
    case EPI_SILU_VEC: return for_gemm_variant<false, EPI_SILU_VEC>(idx, f);
    case EPI_STORE_F32: return for_gemm_variant<false, EPI_STORE_F32>(idx, f);
    case EPI_RESID_NORM: return for_gemm_variant<false, EPI_RESID_NORM>(idx, f);
    case EPI_EMBED_NORM: return for_gemm_variant<false, EPI_EMBED_NORM>(idx, f);
    case EPI_STORE_PLANES: return for_gemm_variant<false, EPI_STORE_PLANES>(idx, f);
    default: return cudaErrorInvalidValue;
  }
}

// (function attributes are per device: set once for every device that a handle or a test aid uses)
static cudaError_t ensure_smem_attr() {
  static bool done_dev[64] = {};
  int dev = 0;
  cudaError_t ed = cudaGetDevice(&dev);
  if (ed != cudaSuccess) return ed;
  bool unused = false;
  bool& done = (dev >= 0 && dev < 64) ? done_dev[dev] : unused;
  if (done) return cudaSuccess;
  const int epis[7] = {EPI_STORE, EPI_SILU_VEC, EPI_STORE_F32, EPI_RESID_NORM, EPI_EMBED_NORM, EPI_GEGLU, EPI_STORE_PLANES};
  for (int e6 = 0; e6 < 7; ++e6)
    for (int idx = 0; idx < 16; ++idx) {
      cudaError_t e = for_gemm_kernel(e6 == 5, epis[e6], idx, [](auto kern) {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET + 1024);
      });
      if (e != cudaSuccess) return e;
    }
  for (int e6 = 0; e6 < 6; ++e6)
    for (int idx = 0; idx < 4; ++idx) {
      cudaError_t e = for_pair_kernel(e6 == 5, epis[e6], idx, [](auto kern) {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET + 1024);
      });
      if (e != cudaSuccess) return e;
    }
  done = true;
  return cudaSuccess;
}

static int gemm_grid(const GemmPlan& p, int budget) {
  if (p.pair) {  // pairs of blocks; a pair needs two SMs, so a budget of one is served with two
    const int items = ((p.n_ftiles + 1) / 2) * p.n_ttiles;
    int pairs = budget / 2;
    if (pairs < 1) pairs = 1;
    if (pairs > items) pairs = items;
    return 2 * pairs;
  }
  const int items = p.n_ftiles * p.n_ttiles;
  int clusters = budget / p.splits;
  if (clusters < 1) clusters = 1;
  if (clusters > items) clusters = items;
  return clusters * p.splits;
}

// Enqueue one projection: clusters of p.splits blocks, at most `budget` blocks in total.
static cudaError_t launch_gemm(const CUtensorMap& map_w, const CUtensorMap& map_a, const GemmPlan& p, bool dual,
                               GemmArgs g, int budget, cudaStream_t st, bool pdl = false) {
  g.kb_total = p.kb_total; g.tile_tok = p.tile_tok; g.n_ftiles = p.n_ftiles; g.n_ttiles = p.n_ttiles;
  g.splits = p.splits; g.stages = p.stages; g.tmem_cols = p.tmem_cols; g.ring_bytes = p.ring_bytes;
  g.acc_bufs = p.acc_bufs; g.issuers = p.issuers;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)gemm_grid(p, budget));
  cfg.blockDim = dim3(GEMM_THREADS);
  cfg.dynamicSmemBytes = p.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (p.splits > 1 || p.pair) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = p.pair ? 2u : (unsigned)p.splits;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  // tokens per epilogue chunk: 32 for wide tiles that are a multiple of 32, else 16
  const bool wide = (p.tile_tok & 31) == 0 && p.tile_tok >= 96;
  if (p.pair)
    return for_pair_kernel(dual, g.epi, (wide ? 1 : 0) | ((g.dbg || g.trace) ? 2 : 0),
                           [&](auto kern) { return cudaLaunchKernelEx(&cfg, kern, map_w, map_a, g); });
  const int idx = (wide ? 1 : 0) | (p.splits > 1 ? 2 : 0) | (p.issuers == 2 ? 4 : 0) | ((g.dbg || g.trace) ? 8 : 0);
  return for_gemm_kernel(dual, g.epi, idx, [&](auto kern) { return cudaLaunchKernelEx(&cfg, kern, map_w, map_a, g); });
}

}  // namespace tc
}  // namespace adit
