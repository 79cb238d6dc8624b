// Host side of the ADiT library: handle, validation, weight repacking and the launch plan of
// adit_denoise.  Everything behind the C ABI declared in include/adit.h.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <tuple>
#include <cstdlib>
#include <vector>

#include "../../include/adit.h"
#include "common.cuh"
#include "ref_kernels.cuh"
#include "tc_host.cuh"
#include "attention.cuh"
#include "attention_tc.cuh"
#include "tc_aux_kernels.cuh"
#include "loop_kernel.cuh"
#include <mutex>

using namespace adit;

#define CU_TRY(h, expr)                                   \
  do {                                                    \
    cudaError_t e_ = (expr);                              \
    if (e_ != cudaSuccess) {                              \
      if (h) (h)->last_cuda = (int)e_;                    \
      return ADIT_E_CUDA;                                 \
    }                                                     \
  } while (0)

struct LayerWeights {
  void *wqkv, *wo, *wgu, *wd;  // compute dtype, [out, in] row-major (in contiguous)
  CUtensorMap m_qkv, m_o, m_gu, m_d;  // TMA descriptors of the above (tensor-core path)
};

struct adit_handle {
  adit_config cfg;
  int device = 0, sm_count = 0;
  bool loaded = false;
  int n_tok = 0;       // suffix tokens per request
  int gu_block = 0;    // gate/up row interleave block
  size_t esz = 4;      // bytes per compute-dtype element
  std::map<std::string, float*> raw;  // staged fp32 copies until every tensor has arrived
  std::vector<void*> allocs;          // everything cudaMalloc'ed for packed weights + workspace
  // packed weights
  float *Wa = 0, *ba = 0, *Ws = 0, *bs = 0, *b1 = 0, *b2 = 0, *Wout = 0, *bout = 0;
  void *W1a = 0, *W1t = 0, *W2 = 0;
  float *Wfold = 0, *bfold = 0;  // action projection folded into the first action-time MLP layer (tensor-core path)
  CUtensorMap m_w1a, m_w2;
  CUtensorMap m_q;     // query rows of the qkv workspace (attention kernel)
  bool q_tma = false;
  std::vector<LayerWeights> layers;
  float *ssq = 0, *rstd_state = 0;  // per-feature-tile sums of squares; the state token's 1/rms (tensor-core path)
  int* counters = 0;                // arrival counters of the norm-statistics epilogue
  bf16* hsb = 0;                    // bf16 copy of the state token rows
  int ctime_steps = 0; // the K for which ctime currently holds the time vectors (tensor-core path)
  CallDesc* desc_dev = 0;          // per-call descriptor read by the kernels of the launch graph
  KvMaps* kvmaps_dev = 0;          // per-call tensor maps of the prefix caches (tensor-core attention)
  CUtensorMap m_sfx;               // this step's K/V rows in the qkv workspace: boxes of 64 rows x 64 channels; its row
  int64_t m_sfx_rows = 0;          //   extent is the call's token count, so rows left by an earlier, larger call read as zeros
  cudaStream_t cap_stream = 0;     // stream used only to capture launch graphs
  bool use_graph = true, use_pdl = true;
  // optional timeline: per launch, every block's start/end timestamp
  bool tracing = false;
  unsigned long long* trace_dev = 0;
  size_t trace_cap = 0, trace_off = 0;  // in uint64 elements
  struct TraceRec { int cls, grid; size_t off; };
  std::vector<TraceRec> trace_recs;
  struct GraphEntry { cudaGraphExec_t exec; int64_t launches; };
  std::map<std::tuple<int, int, int>, GraphEntry> graphs;  // keyed by (B, K, thread-block budget)
  float *att_po = 0, *att_pml = 0;  // key-split partials of the attention kernel
  // workspace
  float *x = 0, *h = 0, *hs = 0, *rstd = 0, *tau = 0, *ctime = 0, *state_dev = 0, *noise_dev = 0;
  void *hb = 0, *qkv = 0, *att = 0, *mlp = 0, *ea = 0, *ez = 0;
  int* status_host = 0;  // pinned, device-visible status word
  int* status_dev = 0;   // its device address
  float2* rope_tab = 0;  // cos/sin per suffix token row and channel pair (variant ADIT_FLAG_SUFFIX_ROPE)
  // hidden-state hand-over (adit_project_prefix): the prefix K/V projections of every layer as one matrix
  void* Wp = 0;                // bf16 [n_layers * 2 * KV, prefix_hidden_dim], rows ordered (layer, K then V, kv head, channel)
  int prefix_hidden_dim = 0;   // 0 until adit_load_prefix_projection has run
  CUtensorMap m_wp;
  int64_t launches = 0;
  int last_cuda = 0;
  bool profiling = false;
  struct ProfRec { int cls; cudaEvent_t a, b; };
  std::vector<ProfRec> prof;
  // persistent small-batch loop (loop_kernel.cuh)
  bool loop_ok = false;            // the shape family and the device can run it
  int loop_clusters = 0;           // clusters of 8 blocks that are resident at once on this device
  CUtensorMap* maps_dev = 0;       // tensor maps of the loop kernel, device memory
  uint32_t* loop_counters = 0;     // level counters + abort word
  uint8_t* loop_scratch = 0;       // per-cluster partial sums of the loop kernel
  loop::GemmLv loop_g[loop::G_COUNT];
  cudaEvent_t loop_ev = 0;         // end of this handle's most recent persistent call
  unsigned long long wait_limit_ns = 2000000000ull;  // bound of every device-side wait of the loop kernel
  int debug_skip_level = -1;       // test aid (adit_debug_wait_limit)
  unsigned long long* loop_trace = 0;  // [levels][blocks][4] timestamps of the most recent call while tracing
  size_t loop_trace_cap = 0;
  int loop_trace_levels = 0, loop_trace_blocks = 0, loop_trace_layers = 0;
};

// Kernel classes for the optional per-launch device timing (adit_profile_*).
enum KernelClass : int {
  KC_PROLOGUE = 0, KC_EMBED, KC_NORM, KC_GEMM_QKV, KC_ATTENTION, KC_GEMM_O, KC_GEMM_GATEUP, KC_GEMM_DOWN,
  KC_FINAL, KC_REDUCE, KC_LOOP, KC_COUNT
};
static_assert(KC_COUNT == ADIT_N_KERNEL_CLASSES, "header and library disagree on the class count");

// Brackets the launches issued during its lifetime with a pair of events when profiling is on.
struct ProfScope {
  adit_handle* h; cudaStream_t st; cudaEvent_t b = nullptr;
  ProfScope(adit_handle* h_, int cls, cudaStream_t st_) : h(h_), st(st_) {
    if (!h->profiling) return;
    cudaEvent_t a;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { b = nullptr; return; }
    cudaEventRecord(a, st);
    h->prof.push_back({cls, a, b});
  }
  ~ProfScope() { if (b) cudaEventRecord(b, st); }
};

static int dev_alloc(adit_handle* h, void** p, size_t bytes) {
  void* q = nullptr;
  CU_TRY(h, cudaMalloc(&q, bytes < 256 ? 256 : bytes));
  h->allocs.push_back(q);
  // Padding rows of the activation buffers are read as MMA operands (their results are discarded): they must hold
  // finite values, never what the allocator left behind.
  CU_TRY(h, cudaMemset(q, 0, bytes < 256 ? 256 : bytes));
  *p = q;
  return ADIT_OK;
}

extern "C" const char* adit_strerror(int code) {
  switch (code) {
    case ADIT_OK: return "ok";
    case ADIT_E_INVALID: return "invalid argument";
    case ADIT_E_CAPACITY: return "capacity exceeded";
    case ADIT_E_NOT_LOADED: return "weights not loaded";
    case ADIT_E_UNSUPPORTED: return "unsupported shape or device";
    case ADIT_E_CUDA: return "CUDA error";
    case ADIT_E_TIMEOUT: return "device wait timed out";
    default: return "unknown status";
  }
}

// Attention launch plan: depends on the batch size and the handle's capacity only, never on the
// per-call SM budget or on the actual prefix lengths, so results do not change with either.
struct AttnPlan { int nw, n_row_tiles, splits; };
static AttnPlan plan_attention(const adit_handle* h, int B) {
  const adit_config& c = h->cfg;
  const int G = c.n_q_heads / c.n_kv_heads, R = h->n_tok * G;
  AttnPlan p;
  p.nw = R <= 32 ? 2 : 4;
  const bool tc_kernel = !(c.flags & ADIT_FLAG_MMA_SYNC_ATTENTION);
  const int rows = tc_kernel ? attn::TC_ROWS : 16 * p.nw;
  p.n_row_tiles = (R + rows - 1) / rows;
  const int base = B * c.n_kv_heads * p.n_row_tiles;
  const int max_nkb = (c.max_prefix_len + h->n_tok + attn::KEY_BLOCK - 1) / attn::KEY_BLOCK;
  p.splits = 1;
  if (base * 10 < h->sm_count * 7) {
    p.splits = tc_kernel ? h->sm_count / base : (h->sm_count + base - 1) / base;  // one wave of blocks
    if (p.splits < 1) p.splits = 1;
    if (p.splits > max_nkb) p.splits = max_nkb;
    if (p.splits > 32) p.splits = 32;  // the merge kernel keeps one split per lane
  }
  return p;
}

// Writes the call's prefix-cache tensor maps to device memory (they arrive as a by-value parameter, so the caller's
// host arrays are consumed at enqueue time) and releases them to the copy engine's proxy.
__global__ void set_kvmaps_kernel(const __grid_constant__ KvMaps m, KvMaps* __restrict__ dst, int n) {
  const uint4* src = reinterpret_cast<const uint4*>(&m);
  uint4* d = reinterpret_cast<uint4*>(dst);
  for (int i = threadIdx.x; i < n * (int)(sizeof(CUtensorMap) / 16); i += blockDim.x) d[i] = src[i];
  __syncthreads();
  if (threadIdx.x == 0) ptx::tensormap_release();
}

struct LoopInFlight { adit_handle* h; int device; cudaEvent_t ev; int clusters; };
static std::mutex g_loop_mutex;
static std::vector<LoopInFlight> g_loop_inflight;
static bool stream_is_capturing(cudaStream_t st) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  return cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusActive;
}
static cudaError_t init_attention_attrs();
static int loop_init(adit_handle* h);
static bool make_map_prefix(CUtensorMap* m, const void* base, int dh, int plen, int p_cap, int64_t planes);
static int loop_build_maps(adit_handle* h);
static const int ROW_PAD = 320;  // rows beyond the last token that a token tile (<= 256 wide, remapped rows) may touch
static bool use_reference_kernels(const adit_config& c) {
  return c.dtype == ADIT_DTYPE_FP32 || (c.flags & ADIT_FLAG_REFERENCE_KERNELS);
}

static int validate_config(const adit_config* c) {
  if (!c) return ADIT_E_INVALID;
  if (c->n_layers < 1 || c->d_model < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->head_dim < 1 ||
      c->d_ff < 1 || c->horizon < 1 || c->action_dim < 1 || c->state_dim < 1 || c->time_emb_dim < 4 ||
      c->max_batch < 1 || c->max_prefix_len < 0)
    return ADIT_E_INVALID;
  if (c->n_q_heads % c->n_kv_heads != 0 || (c->time_emb_dim & 1)) return ADIT_E_INVALID;
  if (c->dtype != ADIT_DTYPE_FP32 && c->dtype != ADIT_DTYPE_BF16) return ADIT_E_INVALID;
  if (!(c->rms_eps >= 0.f) || !(c->t_min_period > 0.f) || !(c->t_max_period > 0.f)) return ADIT_E_INVALID;
  if (c->max_batch > ADIT_MAX_BATCH) return ADIT_E_CAPACITY;
  if (c->head_dim != 64 && c->head_dim != 128 && c->head_dim != 256) return ADIT_E_UNSUPPORTED;
  if (c->d_model % 4) return ADIT_E_UNSUPPORTED;
  if ((c->flags & ADIT_FLAG_STATE_BLOCK_MASK) && (c->flags & ADIT_FLAG_MMA_SYNC_ATTENTION)) return ADIT_E_UNSUPPORTED;
  if (!use_reference_kernels(*c)) {
    if (c->d_model % 64 || c->d_ff % 64) return ADIT_E_UNSUPPORTED;
  }
  return ADIT_OK;
}

extern "C" int adit_create(const adit_config* cfg, int device, adit_handle** out) {
  if (!out) return ADIT_E_INVALID;
  int rc = validate_config(cfg);
  if (rc) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return ADIT_E_INVALID;
  adit_handle* h = new (std::nothrow) adit_handle();
  if (!h) return ADIT_E_INVALID;
  h->cfg = *cfg;
  h->device = device;
  auto fail = [&](int code) {
    adit_destroy(h);
    return code;
  };
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return fail(ADIT_E_CUDA);
  if (!use_reference_kernels(*cfg) && prop.major != 10) return fail(ADIT_E_UNSUPPORTED);
  h->sm_count = prop.multiProcessorCount;
  if (cudaSetDevice(device) != cudaSuccess) return fail(ADIT_E_CUDA);
  const adit_config& c = h->cfg;
  h->n_tok = 1 + c.horizon;
  h->esz = c.dtype == ADIT_DTYPE_BF16 ? 2 : 4;
  h->gu_block = (c.d_ff % 128 == 0) ? 128 : c.d_ff;
  const int64_t D = c.d_model, F = c.d_ff, Q = (int64_t)c.n_q_heads * c.head_dim,
                KV = (int64_t)c.n_kv_heads * c.head_dim, A = c.action_dim, S = c.state_dim, T = c.time_emb_dim;
  // activation buffers carry ROW_PAD extra rows: the tensor-core epilogues store whole token tiles
  const int64_t Mx = (int64_t)c.max_batch * h->n_tok + ROW_PAD, Ma = (int64_t)c.max_batch * c.horizon + ROW_PAD;
  const size_t e = h->esz;
#define ALLOC(ptr, bytes)                                            \
  do {                                                               \
    int rc_ = dev_alloc(h, (void**)&(ptr), (size_t)(bytes));         \
    if (rc_) return fail(rc_);                                       \
  } while (0)
  ALLOC(h->Wa, D * A * 4); ALLOC(h->ba, D * 4); ALLOC(h->Ws, D * S * 4); ALLOC(h->bs, D * 4);
  ALLOC(h->b1, D * 4); ALLOC(h->b2, D * 4); ALLOC(h->Wout, A * D * 4); ALLOC(h->bout, A * 4);
  ALLOC(h->W1a, D * D * e); ALLOC(h->W1t, D * T * e); ALLOC(h->W2, D * D * e);
  ALLOC(h->Wfold, D * A * 4); ALLOC(h->bfold, D * 4);
  h->layers.resize(c.n_layers);
  for (auto& L : h->layers) {
    ALLOC(L.wqkv, (Q + 2 * KV) * D * e); ALLOC(L.wo, D * Q * e);
    ALLOC(L.wgu, 2 * F * D * e); ALLOC(L.wd, D * F * e);
  }
  ALLOC(h->x, Ma * A * 4); ALLOC(h->h, Mx * D * 4); ALLOC(h->hs, c.max_batch * D * 4);
  ALLOC(h->rstd, Mx * 4); ALLOC(h->tau, (int64_t)ADIT_MAX_STEPS * T * 4);
  ALLOC(h->ctime, (int64_t)ADIT_MAX_STEPS * D * 4);
  ALLOC(h->state_dev, c.max_batch * S * 4); ALLOC(h->noise_dev, Ma * A * 4);
  ALLOC(h->hb, Mx * D * e); ALLOC(h->qkv, Mx * (Q + 2 * KV) * e); ALLOC(h->att, Mx * Q * e);
  ALLOC(h->mlp, Mx * F * e); ALLOC(h->ea, Ma * D * e); ALLOC(h->ez, Ma * D * e);
  if (c.flags & ADIT_FLAG_SUFFIX_ROPE) ALLOC(h->rope_tab, Mx * (c.head_dim / 2) * 8);
  if (!use_reference_kernels(c)) {
    const int64_t n_ft = (D + tc::TILE_F - 1) / tc::TILE_F;
    ALLOC(h->ssq, n_ft * Mx * 4);
    ALLOC(h->counters, Mx * 4);
    ALLOC(h->rstd_state, c.max_batch * 4);
    ALLOC(h->hsb, c.max_batch * D * 2);
    if (cudaMemset(h->counters, 0, Mx * 4) != cudaSuccess) return fail(ADIT_E_CUDA);
    if (tc::ensure_smem_attr() != cudaSuccess || !tc::encode_tiled_fn()) return fail(ADIT_E_CUDA);
    if (c.d_ff % 128) return fail(ADIT_E_UNSUPPORTED);
    int64_t worst = 1;
    for (int b = 1; b <= c.max_batch; ++b) {
      AttnPlan ap = plan_attention(h, b);
      int64_t rows = ap.splits > 1 ? (int64_t)ap.splits * b * h->n_tok * c.n_q_heads : 0;
      if (rows > worst) worst = rows;
    }
    ALLOC(h->att_po, worst * c.head_dim * 4);
    ALLOC(h->att_pml, worst * 2 * 4);
    ALLOC(h->desc_dev, sizeof(CallDesc));
    ALLOC(h->kvmaps_dev, sizeof(KvMaps));
    if (!tc::make_map_bf16(&h->m_sfx, h->qkv, (uint64_t)Mx, (uint64_t)(Q + 2 * KV), attn::KEY_BLOCK)) return fail(ADIT_E_CUDA);
    h->m_sfx_rows = Mx;
    h->q_tma = tc::make_map_q(&h->m_q, h->qkv, (uint64_t)Mx, (uint64_t)(Q + 2 * KV), (uint32_t)c.head_dim,
                              (uint32_t)c.n_q_heads, (uint32_t)(c.n_q_heads / c.n_kv_heads));
    if (!h->q_tma) memset(&h->m_q, 0, sizeof(h->m_q));
    if (cudaStreamCreateWithFlags(&h->cap_stream, cudaStreamNonBlocking) != cudaSuccess) return fail(ADIT_E_CUDA);
    if (init_attention_attrs() != cudaSuccess) return fail(ADIT_E_CUDA);
    h->use_graph = !(c.flags & ADIT_FLAG_NO_GRAPH);
    h->use_pdl = !(c.flags & ADIT_FLAG_NO_PDL);
    int rc_loop = loop_init(h);
    if (rc_loop) return fail(rc_loop);
  }
#undef ALLOC
  if (cudaHostAlloc((void**)&h->status_host, sizeof(int), cudaHostAllocMapped) != cudaSuccess)
    return fail(ADIT_E_CUDA);
  *h->status_host = 0;
  if (cudaHostGetDevicePointer((void**)&h->status_dev, h->status_host, 0) != cudaSuccess) return fail(ADIT_E_CUDA);
  *out = h;
  return ADIT_OK;
}

extern "C" int adit_destroy(adit_handle* h) {
  if (!h) return ADIT_OK;
  cudaSetDevice(h->device);
  cudaDeviceSynchronize();
  {
    std::lock_guard<std::mutex> lock(g_loop_mutex);
    for (auto it = g_loop_inflight.begin(); it != g_loop_inflight.end();)
      it = it->h == h ? g_loop_inflight.erase(it) : it + 1;
  }
  if (h->loop_ev) cudaEventDestroy(h->loop_ev);
  for (auto& g : h->graphs) cudaGraphExecDestroy(g.second.exec);
  if (h->cap_stream) cudaStreamDestroy(h->cap_stream);
  for (void* p : h->allocs) cudaFree(p);
  for (auto& kv : h->raw) cudaFree(kv.second);
  if (h->status_host) cudaFreeHost(h->status_host);
  delete h;
  return ADIT_OK;
}

extern "C" int adit_poll_status(adit_handle* h) {
  if (!h) return ADIT_E_INVALID;
  return *(volatile int*)h->status_host;
}
extern "C" int adit_last_cuda_error(adit_handle* h) { return h ? h->last_cuda : 0; }
extern "C" int64_t adit_kernel_launches(adit_handle* h) { return h ? h->launches : 0; }

// ---------------------------------------------------------------------------------------------
// Weight loading
// ---------------------------------------------------------------------------------------------
static bool expected_shape(const adit_config& c, const std::string& name, int* ndim, int64_t shape[2]) {
  const int64_t D = c.d_model, F = c.d_ff, Q = (int64_t)c.n_q_heads * c.head_dim,
                KV = (int64_t)c.n_kv_heads * c.head_dim, A = c.action_dim, S = c.state_dim, T = c.time_emb_dim;
  auto set2 = [&](int64_t a, int64_t b) { *ndim = 2; shape[0] = a; shape[1] = b; return true; };
  auto set1 = [&](int64_t a) { *ndim = 1; shape[0] = a; shape[1] = 1; return true; };
  if (name == "action_in.w") return set2(A, D);
  if (name == "action_in.b") return set1(D);
  if (name == "state_in.w") return set2(S, D);
  if (name == "state_in.b") return set1(D);
  if (name == "time_mlp.w1") return set2(D + T, D);
  if (name == "time_mlp.b1") return set1(D);
  if (name == "time_mlp.w2") return set2(D, D);
  if (name == "time_mlp.b2") return set1(D);
  if (name == "final_norm.g") return set1(D);
  if (name == "action_out.w") return set2(D, A);
  if (name == "action_out.b") return set1(A);
  if (name.rfind("layers.", 0) == 0) {
    size_t dot = name.find('.', 7);
    if (dot == std::string::npos || dot == 7) return false;
    for (size_t i = 7; i < dot; ++i)
      if (name[i] < '0' || name[i] > '9') return false;
    long l = strtol(name.substr(7, dot - 7).c_str(), nullptr, 10);
    if (l < 0 || l >= c.n_layers) return false;
    std::string leaf = name.substr(dot + 1);
    if (leaf == "norm1.g" || leaf == "norm2.g") return set1(D);
    if (leaf == "wq") return set2(D, Q);
    if (leaf == "wk" || leaf == "wv") return set2(D, KV);
    if (leaf == "wo") return set2(Q, D);
    if (leaf == "wg" || leaf == "wu") return set2(D, F);
    if (leaf == "wd") return set2(F, D);
  }
  return false;
}

static size_t n_expected_tensors(const adit_config& c) { return 11 + 9 * (size_t)c.n_layers; }

template <typename T>
static void pack(adit_handle* h, const std::string& src, const char* gain, void* dst, int64_t row_off, int n_in,
                 int n_out, int ld, int gu_block = 0, int gu_second = 0) {
  int64_t n = (int64_t)n_in * n_out;
  pack_rows_kernel<T><<<(unsigned)((n + 255) / 256), 256>>>(h->raw[src], n_in, n_out, gain ? h->raw[gain] : nullptr,
                                                           (T*)dst, row_off, ld, gu_block, gu_second);
}

template <typename T>
static int pack_all(adit_handle* h) {
  const adit_config& c = h->cfg;
  const int D = c.d_model, F = c.d_ff, Q = c.n_q_heads * c.head_dim, KV = c.n_kv_heads * c.head_dim,
            A = c.action_dim, S = c.state_dim, Tm = c.time_emb_dim;
  pack<float>(h, "action_in.w", nullptr, h->Wa, 0, A, D, A);
  pack<float>(h, "state_in.w", nullptr, h->Ws, 0, S, D, S);
  pack<float>(h, "action_out.w", "final_norm.g", h->Wout, 0, D, A, D);
  cudaMemcpy(h->ba, h->raw["action_in.b"], D * 4, cudaMemcpyDeviceToDevice);
  cudaMemcpy(h->bs, h->raw["state_in.b"], D * 4, cudaMemcpyDeviceToDevice);
  cudaMemcpy(h->b1, h->raw["time_mlp.b1"], D * 4, cudaMemcpyDeviceToDevice);
  cudaMemcpy(h->b2, h->raw["time_mlp.b2"], D * 4, cudaMemcpyDeviceToDevice);
  cudaMemcpy(h->bout, h->raw["action_out.b"], A * 4, cudaMemcpyDeviceToDevice);
  // time_mlp.w1 is [D + Tm, D]: the first D input rows act on the action embedding, the rest on tau.
  {
    const float* w1 = h->raw["time_mlp.w1"];
    int64_t n = (int64_t)D * D;
    pack_rows_kernel<T><<<(unsigned)((n + 255) / 256), 256>>>(w1, D, D, nullptr, (T*)h->W1a, 0, D, 0, 0);
    n = (int64_t)Tm * D;
    pack_rows_kernel<T><<<(unsigned)((n + 255) / 256), 256>>>(w1 + (int64_t)D * D, Tm, D, nullptr, (T*)h->W1t, 0, Tm,
                                                             0, 0);
  }
  pack<T>(h, "time_mlp.w2", nullptr, h->W2, 0, D, D, D);
  for (int l = 0; l < c.n_layers; ++l) {
    std::string p = "layers." + std::to_string(l) + ".";
    std::string g1 = p + "norm1.g", g2 = p + "norm2.g";
    LayerWeights& L = h->layers[l];
    pack<T>(h, p + "wq", g1.c_str(), L.wqkv, 0, D, Q, D);
    pack<T>(h, p + "wk", g1.c_str(), L.wqkv, Q, D, KV, D);
    pack<T>(h, p + "wv", g1.c_str(), L.wqkv, Q + KV, D, KV, D);
    pack<T>(h, p + "wo", nullptr, L.wo, 0, Q, D, Q);
    pack<T>(h, p + "wg", g2.c_str(), L.wgu, 0, D, F, D, h->gu_block, 0);
    pack<T>(h, p + "wu", g2.c_str(), L.wgu, 0, D, F, D, h->gu_block, 1);
    pack<T>(h, p + "wd", nullptr, L.wd, 0, F, D, F);
  }
  CU_TRY(h, cudaGetLastError());
  CU_TRY(h, cudaDeviceSynchronize());
  if (!use_reference_kernels(c)) {
    tc::fold_embed_kernel<<<D, 256>>>((const bf16*)h->W1a, (const float*)h->Wa, (const float*)h->ba, h->Wfold, h->bfold, D, A);
    CU_TRY(h, cudaGetLastError());
    CU_TRY(h, cudaDeviceSynchronize());
    bool ok = tc::make_map_bf16(&h->m_w1a, h->W1a, D, D, tc::TILE_F) && tc::make_map_bf16(&h->m_w2, h->W2, D, D, tc::TILE_F);
    for (auto& L : h->layers) {
      ok = ok && tc::make_map_bf16(&L.m_qkv, L.wqkv, Q + 2 * KV, D, tc::TILE_F) &&
           tc::make_map_bf16(&L.m_o, L.wo, D, Q, tc::TILE_F) &&
           tc::make_map_bf16(&L.m_gu, L.wgu, 2 * F, D, 2 * tc::TILE_F) &&
           tc::make_map_bf16(&L.m_d, L.wd, D, F, tc::TILE_F);
    }
    if (!ok) return ADIT_E_CUDA;
    int rc_maps = loop_build_maps(h);
    if (rc_maps) return rc_maps;
  }
  for (auto& kv : h->raw) cudaFree(kv.second);
  h->raw.clear();
  h->ctime_steps = 0;
  h->loaded = true;
  return ADIT_OK;
}

extern "C" int adit_load_weights(adit_handle* h, const adit_tensor* tensors, int n_tensors) {
  if (!h || (!tensors && n_tensors > 0) || n_tensors < 0) return ADIT_E_INVALID;
  CU_TRY(h, cudaSetDevice(h->device));
  // validate everything first so that an error leaves the handle as it was
  for (int i = 0; i < n_tensors; ++i) {
    const adit_tensor& t = tensors[i];
    if (!t.name || !t.data) return ADIT_E_INVALID;
    int nd;
    int64_t shp[2];
    if (!expected_shape(h->cfg, t.name, &nd, shp)) return ADIT_E_INVALID;
    if (t.ndim != nd || t.shape[0] != shp[0] || (nd == 2 && t.shape[1] != shp[1])) return ADIT_E_INVALID;
    if (t.dtype != ADIT_DTYPE_FP32 && t.dtype != ADIT_DTYPE_BF16) return ADIT_E_INVALID;
  }
  if (h->loaded && n_tensors > 0) h->loaded = false;  // a reload replaces tensors; repack when complete
  for (int i = 0; i < n_tensors; ++i) {
    const adit_tensor& t = tensors[i];
    int nd;
    int64_t shp[2];
    expected_shape(h->cfg, t.name, &nd, shp);
    int64_t n = shp[0] * shp[1];
    float* dst = nullptr;
    auto it = h->raw.find(t.name);
    if (it != h->raw.end()) dst = it->second;
    else {
      CU_TRY(h, cudaMalloc((void**)&dst, (size_t)n * 4));
      h->raw[t.name] = dst;
    }
    cudaMemcpyKind kind = t.on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    if (t.dtype == ADIT_DTYPE_FP32) {
      CU_TRY(h, cudaMemcpy(dst, t.data, (size_t)n * 4, kind));
    } else {
      uint16_t* tmp = nullptr;
      CU_TRY(h, cudaMalloc((void**)&tmp, (size_t)n * 2));
      cudaError_t e = cudaMemcpy(tmp, t.data, (size_t)n * 2, kind);
      if (e == cudaSuccess) {
        bf16_bits_to_f32_kernel<<<(unsigned)((n + 255) / 256), 256>>>(tmp, dst, n);
        e = cudaDeviceSynchronize();
      }
      cudaFree(tmp);
      CU_TRY(h, e);
    }
  }
  if (h->raw.size() == n_expected_tensors(h->cfg))
    return h->cfg.dtype == ADIT_DTYPE_BF16 ? pack_all<bf16>(h) : pack_all<float>(h);
  return ADIT_OK;
}

// ---------------------------------------------------------------------------------------------
// Hidden-state hand-over: the expert projects the prefix K/V itself, once per call
// ---------------------------------------------------------------------------------------------
// Copies one tensor to a fresh device buffer as fp32 (the caller frees it).
static int stage_f32(adit_handle* h, const adit_tensor& t, int64_t n, float** out) {
  float* dst = nullptr;
  CU_TRY(h, cudaMalloc((void**)&dst, (size_t)n * 4));
  const cudaMemcpyKind kind = t.on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  cudaError_t e;
  if (t.dtype == ADIT_DTYPE_FP32) {
    e = cudaMemcpy(dst, t.data, (size_t)n * 4, kind);
  } else {
    uint16_t* tmp = nullptr;
    e = cudaMalloc((void**)&tmp, (size_t)n * 2);
    if (e == cudaSuccess) e = cudaMemcpy(tmp, t.data, (size_t)n * 2, kind);
    if (e == cudaSuccess) {
      bf16_bits_to_f32_kernel<<<(unsigned)((n + 255) / 256), 256>>>(tmp, dst, n);
      e = cudaDeviceSynchronize();
    }
    if (tmp) cudaFree(tmp);
  }
  if (e != cudaSuccess) { cudaFree(dst); h->last_cuda = (int)e; return ADIT_E_CUDA; }
  *out = dst;
  return ADIT_OK;
}

extern "C" int adit_load_prefix_projection(adit_handle* h, const adit_tensor* tensors, int n_tensors) {
  if (!h || !tensors) return ADIT_E_INVALID;
  const adit_config& c = h->cfg;
  if (use_reference_kernels(c)) return ADIT_E_UNSUPPORTED;  // (tensor-core path only)
  if (c.flags & ADIT_FLAG_SUFFIX_ROPE) return ADIT_E_UNSUPPORTED;  // (prefix keys would need their own rotation)
  const int L = c.n_layers, KV = c.n_kv_heads * c.head_dim;
  if (n_tensors != 2 * L) return ADIT_E_INVALID;
  // every layer's prefix_wk and prefix_wv exactly once, all [Dh, KV] with one Dh that is a multiple of 64
  std::vector<int> slot(2 * L, -1);
  int64_t Dh = 0;
  for (int i = 0; i < n_tensors; ++i) {
    const adit_tensor& t = tensors[i];
    if (!t.name || !t.data || t.ndim != 2 || t.shape[1] != KV) return ADIT_E_INVALID;
    if (t.dtype != ADIT_DTYPE_FP32 && t.dtype != ADIT_DTYPE_BF16) return ADIT_E_INVALID;
    const std::string name = t.name;
    if (name.rfind("layers.", 0) != 0) return ADIT_E_INVALID;
    const size_t dot = name.find('.', 7);
    if (dot == std::string::npos || dot == 7) return ADIT_E_INVALID;
    for (size_t k = 7; k < dot; ++k)
      if (name[k] < '0' || name[k] > '9') return ADIT_E_INVALID;
    const long l = strtol(name.substr(7, dot - 7).c_str(), nullptr, 10);
    const std::string leaf = name.substr(dot + 1);
    if (l < 0 || l >= L || (leaf != "prefix_wk" && leaf != "prefix_wv")) return ADIT_E_INVALID;
    const int s = (int)l * 2 + (leaf == "prefix_wv" ? 1 : 0);
    if (slot[s] >= 0) return ADIT_E_INVALID;
    slot[s] = i;
    if (Dh == 0) Dh = t.shape[0];
    if (t.shape[0] != Dh) return ADIT_E_INVALID;
  }
  if (Dh < 64 || (Dh % 64) || Dh > (1 << 20)) return ADIT_E_INVALID;
  CU_TRY(h, cudaSetDevice(h->device));
  CU_TRY(h, cudaDeviceSynchronize());  // (a call still using the previous matrix has finished)
  void* wp = nullptr;
  CU_TRY(h, cudaMalloc(&wp, (size_t)2 * L * KV * Dh * 2));
  for (int s = 0; s < 2 * L; ++s) {
    float* src = nullptr;
    int rc = stage_f32(h, tensors[slot[s]], Dh * KV, &src);
    if (rc) { cudaFree(wp); return rc; }
    const int64_t n = Dh * KV;
    // [in = Dh, out = KV] -> rows s * KV .. of the [out, in] matrix
    pack_rows_kernel<bf16><<<(unsigned)((n + 255) / 256), 256>>>(src, (int)Dh, KV, nullptr, (bf16*)wp, (int64_t)s * KV, (int)Dh, 0, 0);
    cudaError_t e = cudaDeviceSynchronize();
    cudaFree(src);
    if (e != cudaSuccess) { cudaFree(wp); h->last_cuda = (int)e; return ADIT_E_CUDA; }
  }
  if (!tc::make_map_bf16(&h->m_wp, wp, (uint64_t)2 * L * KV, (uint64_t)Dh, tc::TILE_F)) { cudaFree(wp); return ADIT_E_CUDA; }
  if (h->Wp) {
    for (auto& q : h->allocs)
      if (q == h->Wp) { cudaFree(q); q = nullptr; }
  }
  h->allocs.push_back(wp);
  h->Wp = wp;
  h->prefix_hidden_dim = (int)Dh;
  return ADIT_OK;
}

extern "C" int adit_project_prefix(adit_handle* h, int B, const void* const* hidden, const int32_t* prefix_len,
                                   void* const* prefix_kv_out, int sm_budget, void* stream) {
  if (!h || !hidden || !prefix_len || !prefix_kv_out || B < 1) return ADIT_E_INVALID;
  const adit_config& c = h->cfg;
  if (B > c.max_batch) return ADIT_E_CAPACITY;
  if (!h->Wp) return ADIT_E_NOT_LOADED;
  for (int b = 0; b < B; ++b) {
    if (prefix_len[b] < 0 || prefix_len[b] > c.max_prefix_len) return ADIT_E_INVALID;
    if (prefix_len[b] > 0 && (!hidden[b] || !prefix_kv_out[b])) return ADIT_E_INVALID;
    if (((uintptr_t)hidden[b] & 15) || ((uintptr_t)prefix_kv_out[b] & 15)) return ADIT_E_INVALID;
  }
  CU_TRY(h, cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)stream;
  const int L = c.n_layers, KV = c.n_kv_heads * c.head_dim, Dh = h->prefix_hidden_dim, NF = 2 * L * KV;
  const int G = (sm_budget <= 0 || sm_budget >= h->sm_count) ? h->sm_count : sm_budget;
  for (int b = 0; b < B; ++b) {
    const int P = prefix_len[b];
    if (P == 0) continue;
    // one product per request: [P, Dh] x [NF, Dh]^T, written straight into the cache's planes.  The plan depends on
    // this request's length and the device only, so a request's cache never depends on its neighbours.
    const tc::GemmPlan p = tc::plan_gemm(P, NF, Dh, false, h->sm_count, true);
    CUtensorMap ma;
    if (!tc::make_map_bf16(&ma, hidden[b], (uint64_t)P, (uint64_t)Dh, p.tile_tok)) return ADIT_E_CUDA;
    tc::GemmArgs g{};
    g.n_feat = NF; g.n_tok = P; g.epi = tc::EPI_STORE_PLANES; g.out = prefix_kv_out[b];
    g.plane_w = c.head_dim; g.plane_stride = (int64_t)c.max_prefix_len * c.head_dim;
    g.status = h->status_dev;
    ProfScope ps(h, KC_PROLOGUE, st);
    CU_TRY(h, tc::launch_gemm(h->m_wp, ma, p, false, g, G, st, false));
    h->launches++;
  }
  return ADIT_OK;
}

// ---------------------------------------------------------------------------------------------
// The denoising loop
// ---------------------------------------------------------------------------------------------
template <typename TA, typename TW, typename TO, int EPI, bool DUAL>
static void launch_ref_gemm(adit_handle* h, int cls, cudaStream_t st, const TA* A, int lda, const TW* W, int ldw, int M, int N,
                            int K, EpiArgs ea) {
  ProfScope ps(h, cls, st);
  dim3 grid((N + 63) / 64, (M + 63) / 64);
  ref_gemm_kernel<TA, TW, TO, EPI, DUAL><<<grid, 256, 0, st>>>(A, lda, W, ldw, DUAL ? h->gu_block : 0,
                                                              DUAL ? h->gu_block : 1, M, N, K, ea);
  h->launches++;
}

template <typename T>
static void launch_ref_attention(adit_handle* h, cudaStream_t st, const PrefixTable& pt, int layer, int B) {
  const adit_config& c = h->cfg;
  const int Q = c.n_q_heads * c.head_dim, QKV = Q + 2 * c.n_kv_heads * c.head_dim;
  ProfScope ps(h, KC_ATTENTION, st);
  dim3 grid(h->n_tok, c.n_q_heads, B);
  const float scale = 1.0f / sqrtf((float)c.head_dim);
#define LAUNCH_ATT(DH)                                                                                        \
  ref_attention_kernel<T, DH><<<grid, 128, 0, st>>>((const T*)h->qkv, QKV, (T*)h->att, Q, pt, layer, h->n_tok, \
                                                    c.n_q_heads, c.n_kv_heads, c.max_prefix_len, scale,       \
                                                    (c.flags & ADIT_FLAG_STATE_BLOCK_MASK) ? 1 : 0)
  if (c.head_dim == 64) LAUNCH_ATT(64);
  else if (c.head_dim == 128) LAUNCH_ATT(128);
  else LAUNCH_ATT(256);
#undef LAUNCH_ATT
  h->launches++;
}

// Plain-kernel loop (fp32 debug path; also bf16 with ADIT_FLAG_REFERENCE_KERNELS).
template <typename T>
static int denoise_reference(adit_handle* h, int B, const PrefixTable& pt, const float* state, const float* noise,
                             int K, cudaStream_t st, float* out) {
  const adit_config& c = h->cfg;
  const int D = c.d_model, F = c.d_ff, Q = c.n_q_heads * c.head_dim, KV = c.n_kv_heads * c.head_dim,
            A = c.action_dim, S = c.state_dim, Tm = c.time_emb_dim, Ta = c.horizon;
  const int M = B * h->n_tok, Ma = B * Ta, QKV = Q + 2 * KV;
  {
    ProfScope ps(h, KC_PROLOGUE, st);
    int n = K * (Tm / 2);
    time_table_kernel<<<(n + 127) / 128, 128, 0, st>>>(h->tau, K, Tm, (double)c.t_min_period, (double)c.t_max_period);
    int n2 = Ma * A > B * D ? Ma * A : B * D;
    prologue_kernel<<<(n2 + 255) / 256, 256, 0, st>>>(nullptr, noise, h->x, Ma * A, state, h->Ws, h->bs, h->hs, B, S, D);
    h->launches += 2;
  }
  {
    // c_k = tau(t_k) . W1[D:, :] + b1 for all k (does not depend on x or the batch)
    launch_ref_gemm<float, T, float, EPI_STORE_F32, false>(h, KC_PROLOGUE, st, h->tau, Tm, (const T*)h->W1t, Tm, K, D, Tm,
                                                           EpiArgs{h->ctime, D, nullptr, h->b1, 0});
  }
  const bool rope = (c.flags & ADIT_FLAG_SUFFIX_ROPE) != 0;
  if (rope) {
    ProfScope ps(h, KC_NORM, st);
    rope_table_kernel<<<(M * (c.head_dim / 2) + 255) / 256, 256, 0, st>>>(h->rope_tab, pt, nullptr, M, h->n_tok, c.head_dim);
    h->launches++;
  }
  const float dt = 1.0f / (float)K;
  for (int k = 0; k < K; ++k) {
    {
      ProfScope ps(h, KC_EMBED, st);
      int64_t n = (int64_t)Ma * D;
      embed_in_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(h->x, h->Wa, h->ba, (T*)h->ea, h->hs, h->h, B,
                                                                       Ta, A, D);
      h->launches++;
    }
    launch_ref_gemm<T, T, T, EPI_SILU_VEC, false>(h, KC_EMBED, st, (const T*)h->ea, D, (const T*)h->W1a, D, Ma, D, D,
                                                  EpiArgs{h->ez, D, nullptr, h->ctime + (int64_t)k * D, 0});
    launch_ref_gemm<T, T, float, EPI_EMBED_OUT, false>(h, KC_EMBED, st, (const T*)h->ez, D, (const T*)h->W2, D, Ma, D, D,
                                                       EpiArgs{h->h, D, nullptr, h->b2, Ta});
    for (int l = 0; l < c.n_layers; ++l) {
      const LayerWeights& L = h->layers[l];
      {
        ProfScope ps(h, KC_NORM, st);
        rowstats_kernel<T><<<M, 256, 0, st>>>(h->h, (T*)h->hb, h->rstd, D, c.rms_eps);
        h->launches++;
      }
      launch_ref_gemm<T, T, T, EPI_STORE, false>(h, KC_GEMM_QKV, st, (const T*)h->hb, D, (const T*)L.wqkv, D, M, QKV, D,
                                                 EpiArgs{h->qkv, QKV, h->rstd, nullptr, 0});
      if (rope) {
        ProfScope ps(h, KC_NORM, st);
        const int nrot = c.n_q_heads + c.n_kv_heads;
        rope_apply_kernel<T><<<(int)(((int64_t)M * nrot * (c.head_dim / 2) + 127) / 128), 128, 0, st>>>((T*)h->qkv, QKV, h->rope_tab, M, nrot,
                                                                                                       c.head_dim);
        h->launches++;
      }
      launch_ref_attention<T>(h, st, pt, l, B);
      launch_ref_gemm<T, T, float, EPI_RESIDUAL, false>(h, KC_GEMM_O, st, (const T*)h->att, Q, (const T*)L.wo, Q, M, D, Q,
                                                        EpiArgs{h->h, D, nullptr, nullptr, 0});
      {
        ProfScope ps(h, KC_NORM, st);
        rowstats_kernel<T><<<M, 256, 0, st>>>(h->h, (T*)h->hb, h->rstd, D, c.rms_eps);
        h->launches++;
      }
      launch_ref_gemm<T, T, T, EPI_GEGLU, true>(h, KC_GEMM_GATEUP, st, (const T*)h->hb, D, (const T*)L.wgu, D, M, F, D,
                                                EpiArgs{h->mlp, F, h->rstd, nullptr, 0});
      launch_ref_gemm<T, T, float, EPI_RESIDUAL, false>(h, KC_GEMM_DOWN, st, (const T*)h->mlp, F, (const T*)L.wd, F, M, D, F,
                                                        EpiArgs{h->h, D, nullptr, nullptr, 0});
    }
    {
      ProfScope ps(h, KC_FINAL, st);
      final_kernel<<<Ma, 256, D * 4, st>>>(h->h, h->Wout, h->bout, h->x, k == K - 1 ? out : nullptr, Ta, A, D,
                                           c.rms_eps, dt, Ma, 1, nullptr);
      h->launches++;
    }
  }
  CU_TRY(h, cudaGetLastError());
  return ADIT_OK;
}

// Reserve a [grid][4] timestamp region for the next launch (null when tracing is off or the buffer is full).
static unsigned long long* trace_slot(adit_handle* h, int cls, int grid) {
  if (!h->tracing || h->trace_off + (size_t)grid * 4 > h->trace_cap) return nullptr;
  unsigned long long* p = h->trace_dev + h->trace_off;
  h->trace_recs.push_back({cls, grid, h->trace_off});
  h->trace_off += (size_t)grid * 4;
  return p;
}

// Launch with (optionally) the programmatic-dependent-launch attribute: the kernel may be scheduled
// while its predecessor in the stream is still running; every kernel of the tensor-core path waits
// (griddepcontrol.wait) before it touches memory the predecessor reads or writes.
template <typename... KArgs, typename... Args>
static cudaError_t launch_k(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, bool pdl,
                            Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// The tcgen05 attention kernel is instantiated per (instrumentation, split key list, query tile by TMA).
template <int DH>
static auto pick_attn_kernel(bool instr, bool partial, bool qtma) -> decltype(&attn::attn_tc_kernel<DH, false, false, true>) {
  const int idx = (instr ? 4 : 0) | (partial ? 2 : 0) | (qtma ? 1 : 0);
  switch (idx) {
    case 0: return attn::attn_tc_kernel<DH, false, false, false>;
    case 1: return attn::attn_tc_kernel<DH, false, false, true>;
    case 2: return attn::attn_tc_kernel<DH, false, true, false>;
    case 3: return attn::attn_tc_kernel<DH, false, true, true>;
    case 4: return attn::attn_tc_kernel<DH, true, false, false>;
    case 5: return attn::attn_tc_kernel<DH, true, false, true>;
    case 6: return attn::attn_tc_kernel<DH, true, true, false>;
    default: return attn::attn_tc_kernel<DH, true, true, true>;
  }
}

template <int DH, int NW>
static cudaError_t attn_attr() {
  return cudaFuncSetAttribute(attn::attn_mma_kernel<DH, NW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)attn::attn_smem_bytes<DH, NW>());
}
static cudaError_t init_attention_attrs() {
  // per device (function attributes belong to a device's copy of the kernel)
  static bool done_dev[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && done_dev[dev]) return cudaSuccess;
  if ((e = attn_attr<64, 2>()) != cudaSuccess) return e;
  if ((e = attn_attr<64, 4>()) != cudaSuccess) return e;
  if ((e = attn_attr<128, 2>()) != cudaSuccess) return e;
  if ((e = attn_attr<128, 4>()) != cudaSuccess) return e;
  if ((e = attn_attr<256, 2>()) != cudaSuccess) return e;
  if ((e = attn_attr<256, 4>()) != cudaSuccess) return e;
#define ADIT_ATTN_ATTR1(DH, IN, PA) \
  if ((e = cudaFuncSetAttribute(attn::attn_tc_kernel<DH, IN, PA, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn::attn_tc_smem_bytes<DH>())) != cudaSuccess) return e; \
  if ((e = cudaFuncSetAttribute(attn::attn_tc_kernel<DH, IN, PA, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn::attn_tc_smem_bytes<DH>())) != cudaSuccess) return e
#define ADIT_ATTN_ATTR(DH, IN) ADIT_ATTN_ATTR1(DH, IN, false); ADIT_ATTN_ATTR1(DH, IN, true)
  ADIT_ATTN_ATTR(64, false); ADIT_ATTN_ATTR(64, true); ADIT_ATTN_ATTR(128, false); ADIT_ATTN_ATTR(128, true);
  ADIT_ATTN_ATTR(256, false); ADIT_ATTN_ATTR(256, true);
#undef ADIT_ATTN_ATTR1
#undef ADIT_ATTN_ATTR
  if (dev >= 0 && dev < 64) done_dev[dev] = true;
  return cudaSuccess;
}

template <int DH>
static void launch_attn_dh(adit_handle* h, const attn::AttnArgs& a_in, const AttnPlan& p, int grid, int merge_grid,
                           int64_t n_qrows, cudaStream_t st) {
  const bool pdl = h->use_pdl;
  attn::AttnArgs a = a_in;
  a.trace = trace_slot(h, KC_ATTENTION, grid);
  a.status = h->status_dev;
  a.kv_maps = h->kvmaps_dev->pk;
  a.q_tma = h->q_tma ? 1 : 0;
  // The last suffix block of the call reaches past its last token: the map ends there, so the copy engine fills those
  // key rows with zeros (their probabilities are zero, but 0 x a stale non-finite value would not be).
  const int64_t rows = (int64_t)a.batch * a.n_tokens;
  if (rows != h->m_sfx_rows && tc::make_map_bf16(&h->m_sfx, h->qkv, (uint64_t)rows, (uint64_t)a.ldqkv, attn::KEY_BLOCK))
    h->m_sfx_rows = rows;
  if (!(h->cfg.flags & ADIT_FLAG_MMA_SYNC_ATTENTION))
    launch_k(pick_attn_kernel<DH>(a.trace != nullptr, a.splits > 1, a.q_tma != 0), grid, attn::TC_THREADS,
             attn::attn_tc_smem_bytes<DH>(), st, pdl, h->m_q, h->m_sfx, a, (const PrefixTable*)&h->desc_dev->pt);
  else if (p.nw == 2)
    launch_k(attn::attn_mma_kernel<DH, 2>, grid, 64, attn::attn_smem_bytes<DH, 2>(), st, pdl, a,
             (const PrefixTable*)&h->desc_dev->pt);
  else
    launch_k(attn::attn_mma_kernel<DH, 4>, grid, 128, attn::attn_smem_bytes<DH, 4>(), st, pdl, a,
             (const PrefixTable*)&h->desc_dev->pt);
  h->launches++;
  if (p.splits > 1) {
    if (!(h->cfg.flags & ADIT_FLAG_MMA_SYNC_ATTENTION))
    {
      // many splits of wide heads: half a row per warp (twice the blocks)
      constexpr int HV = DH >= 128 ? 2 : 1;
      // (a grid capped by the SM budget stays as it is: the kernel strides over its units)
      const int mgrid = (p.splits > 4 && merge_grid == (int)((n_qrows + 3) / 4)) ? merge_grid * HV : merge_grid;
      launch_k(p.splits > 4 ? attn::attn_merge_kernel<DH, bf16, 16, HV> : attn::attn_merge_kernel<DH, bf16, 4>, mgrid, 128, 0,
               st, pdl, (const bf16*)h->att_po, (const float*)h->att_pml, p.splits, n_qrows, h->cfg.n_q_heads,
               (bf16*)h->att, a.ldatt, trace_slot(h, KC_REDUCE, mgrid));
    }
    else
    launch_k(attn::attn_merge_kernel<DH, float>, merge_grid, 128, 0, st, pdl, (const float*)h->att_po,
             (const float*)h->att_pml, p.splits, n_qrows, h->cfg.n_q_heads, (bf16*)h->att, a.ldatt,
             trace_slot(h, KC_REDUCE, merge_grid));
    h->launches++;
  }
}

static void launch_tc_attention(adit_handle* h, cudaStream_t st, int layer, int B, int Gbudget) {
  const adit_config& c = h->cfg;
  const int Q = c.n_q_heads * c.head_dim, QKV = Q + 2 * c.n_kv_heads * c.head_dim;
  ProfScope ps(h, KC_ATTENTION, st);
  AttnPlan p = plan_attention(h, B);
  attn::AttnArgs a{};
  a.qkv = (const bf16*)h->qkv; a.ldqkv = QKV; a.att = (bf16*)h->att; a.ldatt = Q; a.layer = layer;
  a.n_tokens = h->n_tok; a.n_q_heads = c.n_q_heads; a.n_kv_heads = c.n_kv_heads; a.p_cap = c.max_prefix_len;
  a.batch = B; a.n_row_tiles = p.n_row_tiles; a.splits = p.splits;
  a.scale_log2 = 1.4426950408889634f / sqrtf((float)c.head_dim);
  a.part_o = h->att_po; a.part_ml = h->att_pml;
  a.state_mask = (c.flags & ADIT_FLAG_STATE_BLOCK_MASK) ? 1 : 0;
  const int items = B * c.n_kv_heads * p.n_row_tiles * p.splits;
  const bool capped = Gbudget < h->sm_count;
  const int grid = (capped && items > Gbudget) ? Gbudget : items;
  const int64_t n_qrows = (int64_t)B * h->n_tok * c.n_q_heads;
  int mg = (int)((n_qrows + 3) / 4);
  if (capped && mg > Gbudget) mg = Gbudget;
  if (c.head_dim == 64) launch_attn_dh<64>(h, a, p, grid, mg, n_qrows, st);
  else if (c.head_dim == 128) launch_attn_dh<128>(h, a, p, grid, mg, n_qrows, st);
  else launch_attn_dh<256>(h, a, p, grid, mg, n_qrows, st);
}

// Enqueue the whole loop of the tensor-core path on `st` (a user stream, or the capture stream while
// a launch graph is being recorded).  Per-call pointers are read from h->desc_dev on the device.
static int enqueue_tc(adit_handle* h, int B, int K, int G, cudaStream_t st) {
  const adit_config& c = h->cfg;
  const int D = c.d_model, F = c.d_ff, Q = c.n_q_heads * c.head_dim, KV = c.n_kv_heads * c.head_dim,
            A = c.action_dim, S = c.state_dim, Ta = c.horizon;
  const int M = B * h->n_tok, Ma = B * Ta, QKV = Q + 2 * KV;
  const int Mx = c.max_batch * h->n_tok + ROW_PAD, Max = c.max_batch * Ta + ROW_PAD;
  const int SM = h->sm_count;
  const bool pdl = h->use_pdl;
  const bool capped = G < SM;
  h->trace_recs.clear();
  h->trace_off = 0;
  auto cap = [&](int64_t blocks) { return (int)((capped && blocks > G) ? G : blocks); };
  // plans and activation descriptors for this batch size
  const bool two_sm = !(c.flags & ADIT_FLAG_ONE_SM_GEMM);
  tc::GemmPlan p_e2 = tc::plan_projection(Ma, D, D, false, SM, two_sm),
               p_qkv = tc::plan_projection(M, QKV, D, false, SM, two_sm), p_o = tc::plan_projection(M, D, Q, false, SM, two_sm),
               p_gu = tc::plan_projection(M, F, D, true, SM, two_sm), p_d = tc::plan_projection(M, D, F, false, SM, two_sm);
  CUtensorMap a_e2, a_qkv, a_o, a_gu, a_d;
  bool ok = tc::make_map_bf16(&a_e2, h->ez, Max, D, tc::token_box_rows(p_e2)) &&
            tc::make_map_bf16(&a_qkv, h->hb, Mx, D, tc::token_box_rows(p_qkv)) && tc::make_map_bf16(&a_o, h->att, Mx, Q, tc::token_box_rows(p_o)) &&
            tc::make_map_bf16(&a_gu, h->hb, Mx, D, tc::token_box_rows(p_gu)) && tc::make_map_bf16(&a_d, h->mlp, Mx, F, tc::token_box_rows(p_d));
  if (!ok) return ADIT_E_CUDA;

  auto gemm = [&](int cls, const CUtensorMap& mw, const CUtensorMap& ma, const tc::GemmPlan& p, bool dual, int n_tok,
                  int n_feat, int epi, void* outp, int ldo, const float* rowscale, const float* bias) {
    ProfScope ps(h, cls, st);
    tc::GemmArgs g{};
    g.n_feat = n_feat; g.n_tok = n_tok; g.epi = epi; g.out = outp; g.ldo = ldo; g.rowscale = rowscale; g.bias = bias;
    g.h = h->h; g.hb = (bf16*)h->hb; g.ssq = h->ssq; g.ssq_ld = Mx;
    if (rowscale) { g.norm_ssq = h->ssq; g.norm_tiles = (D + tc::TILE_F - 1) / tc::TILE_F; g.norm_dim = D; g.rowscale = nullptr; }
    g.eps = c.rms_eps; g.horizon = Ta; g.status = h->status_dev;
    g.trace = trace_slot(h, cls, tc::gemm_grid(p, G));
    tc::launch_gemm(mw, ma, p, dual, g, G, st, pdl);
    h->launches++;
  };

  {
    ProfScope ps(h, KC_PROLOGUE, st);
    int blocks = (Ma * A + 255) / 256;
    if (blocks < B) blocks = B;
    // first kernel of the sequence: plain stream order behind the descriptor write
    launch_k(tc::prologue_kernel, cap(blocks), 256, 0, st, false, (const CallDesc*)h->desc_dev, h->x, Ma * A,
             (const float*)h->Ws, (const float*)h->bs, h->hs, h->hsb, h->rstd_state, B, S, D);
    h->launches++;
  }
  const bool rope = (c.flags & ADIT_FLAG_SUFFIX_ROPE) != 0;
  if (rope) {
    ProfScope ps(h, KC_NORM, st);
    launch_k(rope_table_kernel, cap((M * (c.head_dim / 2) + 255) / 256), 256, 0, st, pdl, h->rope_tab, PrefixTable{},
             (const PrefixTable*)&h->desc_dev->pt, M, h->n_tok, c.head_dim);
    h->launches++;
  }
  const float dt = 1.0f / (float)K;
  for (int k = 0; k < K; ++k) {
    {
      ProfScope ps(h, KC_EMBED, st);
      const int rpi = Ma >= 512 ? tc::EMB_ROWS : 4;  // rows per work item: fewer for small batches, for more blocks
      const int64_t n = (int64_t)((D + 255) / 256) * ((Ma + rpi - 1) / rpi);  // work items
      launch_k(tc::embed_in_kernel, cap(n > B * ((D + 255) / 256) ? n : B * ((D + 255) / 256)), 256, 0, st, pdl,
               (const float*)h->x, (const float*)h->Wfold, (const float*)h->bfold,
               (const float*)(h->ctime + (int64_t)k * D), (bf16*)h->ez, (const float*)h->hs, (const bf16*)h->hsb,
               (const float*)h->rstd_state, h->h, (bf16*)h->hb, h->ssq, Mx, (D + tc::TILE_F - 1) / tc::TILE_F, B, Ta, A, D, rpi);
      h->launches++;
    }
    gemm(KC_EMBED, h->m_w2, a_e2, p_e2, false, Ma, D, tc::EPI_EMBED_NORM, nullptr, 0, nullptr, h->b2);
    for (int l = 0; l < c.n_layers; ++l) {
      LayerWeights& L = h->layers[l];
      gemm(KC_GEMM_QKV, L.m_qkv, a_qkv, p_qkv, false, M, QKV, EPI_STORE, h->qkv, QKV, h->rstd, nullptr);
      if (rope) {
        ProfScope ps(h, KC_NORM, st);
        const int nrot = c.n_q_heads + c.n_kv_heads;
        launch_k(rope_apply_kernel<bf16>, cap(((int64_t)M * nrot * (c.head_dim / 2) + 127) / 128), 128, 0, st, pdl, (bf16*)h->qkv, QKV,
                 (const float2*)h->rope_tab, M, nrot, c.head_dim);
        h->launches++;
      }
      launch_tc_attention(h, st, l, B, G);
      gemm(KC_GEMM_O, L.m_o, a_o, p_o, false, M, D, tc::EPI_RESID_NORM, nullptr, 0, nullptr, nullptr);
      gemm(KC_GEMM_GATEUP, L.m_gu, a_gu, p_gu, true, M, F, EPI_GEGLU, h->mlp, F, h->rstd, nullptr);
      gemm(KC_GEMM_DOWN, L.m_d, a_d, p_d, false, M, D, tc::EPI_RESID_NORM, nullptr, 0, nullptr, nullptr);
    }
    {
      ProfScope ps(h, KC_FINAL, st);
      const int parts = (Ma < 400 && A >= 32) ? 4 : 1;  // more blocks for small batches
      launch_k(final_kernel, cap((int64_t)Ma * parts), 256, (size_t)D * 4, st, pdl, (const float*)h->h,
               (const float*)h->Wout, (const float*)h->bout, h->x, (float*)nullptr, Ta, A, D, c.rms_eps, dt, Ma, parts,
               (const CallDesc*)(k == K - 1 ? h->desc_dev : nullptr));
      h->launches++;
    }
  }
  if (cudaGetLastError() != cudaSuccess) return ADIT_E_CUDA;
  return ADIT_OK;
}


// ---------------------------------------------------------------------------------------------
// Persistent small-batch loop: plan, tensor maps, launch
// ---------------------------------------------------------------------------------------------

// Launches of the loop kernel that may still be running, per process: two of them whose clusters do not fit the
// device together would each hold part of the SMs and wait for the other's missing blocks.  A call that does not
// fit beside the ones in flight is ordered behind them on the device (an event wait; the host never blocks).

// k-slices per feature tile for one projection: the choice depends on the shape and on the device's cluster
// capacity only (never on the call's SM budget or batch), so the order of every sum is fixed.
static loop::GemmLv plan_loop_gemm(int n_feat, int K, bool dual, int epi, int map_a, int ldo, int clusters_dev) {
  loop::GemmLv g{};
  g.n_ftiles = n_feat / 128;
  g.kb_total = K / 64;
  g.dual = dual ? 1 : 0; g.epi = epi; g.map_a = map_a; g.ldo = ldo;
  double best = 1e30;
  for (int ks = 8; ks >= 2; ks >>= 1) {
    if (g.kb_total % ks) continue;
    const int nf = loop::CS / ks, units = (g.n_ftiles + nf - 1) / nf, kbn = g.kb_total / ks;
    const int rounds = (units + clusters_dev - 1) / clusters_dev;
    const double cost = rounds * (2.0 + 0.035 * kbn * 4 * (dual ? 2 : 1));
    if (cost < best - 1e-9) { best = cost; g.ks = ks; g.nf = nf; g.units = units; g.kbn = kbn; }
  }
  return g;
}

template <int DH>
static cudaError_t loop_prepare_dh(int* clusters) {
  cudaError_t e = cudaFuncSetAttribute(loop::adit_loop_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, loop::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(loop::CS * 64);
  cfg.blockDim = dim3(loop::THREADS);
  cfg.dynamicSmemBytes = loop::SMEM_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = loop::CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(clusters, loop::adit_loop_kernel<DH>, &cfg);
}

// Called from adit_create (tensor-core path): decides whether this shape family and device can run the loop kernel.
static int loop_init(adit_handle* h) {
  const adit_config& c = h->cfg;
  h->loop_ok = false;
  if (!(c.flags & ADIT_FLAG_PERSISTENT_LOOP) || (c.flags & ADIT_FLAG_SUFFIX_ROPE)) return ADIT_OK;
  const int D = c.d_model, F = c.d_ff, Q = c.n_q_heads * c.head_dim, KV = c.n_kv_heads * c.head_dim, QKV = Q + 2 * KV;
  const int G = c.n_q_heads / c.n_kv_heads;
  if (D % 128 || F % 128 || QKV % 128 || Q % 128 || (128 % G) || !h->q_tma) return ADIT_OK;
  if ((D / 64) % 2 || (Q / 64) % 2 || (F / 64) % 2 || D / 128 > 32) return ADIT_OK;
  if (h->n_tok > loop::TOK) return ADIT_OK;
  int clusters = 0;
  cudaError_t e = c.head_dim == 64 ? loop_prepare_dh<64>(&clusters) : c.head_dim == 128 ? loop_prepare_dh<128>(&clusters) : loop_prepare_dh<256>(&clusters);
  if (e != cudaSuccess || clusters < 1) { cudaGetLastError(); return ADIT_OK; }
  h->loop_clusters = clusters;
  h->loop_g[loop::G_W2] = plan_loop_gemm(D, D, false, loop::LEPI_EMBED, loop::MAP_A_EZ, 0, clusters);
  h->loop_g[loop::G_QKV] = plan_loop_gemm(QKV, D, false, loop::LEPI_STORE, loop::MAP_A_HB, QKV, clusters);
  h->loop_g[loop::G_O] = plan_loop_gemm(D, Q, false, loop::LEPI_RESID, loop::MAP_A_ATT, 0, clusters);
  h->loop_g[loop::G_GU] = plan_loop_gemm(F, D, true, loop::LEPI_GEGLU, loop::MAP_A_HB, F, clusters);
  h->loop_g[loop::G_DOWN] = plan_loop_gemm(D, F, false, loop::LEPI_RESID, loop::MAP_A_MLP, 0, clusters);
  for (int i = 0; i < loop::G_COUNT; ++i)
    if (h->loop_g[i].ks == 0) return ADIT_OK;
  void* p = nullptr;
  int rc = dev_alloc(h, &p, sizeof(CUtensorMap) * (size_t)(loop::MAP_LAYER0 + 4 * c.n_layers));
  if (rc) return rc;
  h->maps_dev = (CUtensorMap*)p;
  rc = dev_alloc(h, &p, sizeof(uint32_t) * 2 * loop::LV_COUNT);
  if (rc) return rc;
  h->loop_counters = (uint32_t*)p;
  rc = dev_alloc(h, &p, (size_t)clusters * loop::XS_CLUSTER_BYTES);
  if (rc) return rc;
  h->loop_scratch = (uint8_t*)p;
  CU_TRY(h, cudaEventCreateWithFlags(&h->loop_ev, cudaEventDisableTiming));
  h->loop_ok = true;
  return ADIT_OK;
}

// Called when the weights have been packed: the loop kernel's tensor maps, in device memory.
static int loop_build_maps(adit_handle* h) {
  if (!h->loop_ok) return ADIT_OK;
  const adit_config& c = h->cfg;
  const int64_t D = c.d_model, F = c.d_ff, Q = (int64_t)c.n_q_heads * c.head_dim, KV = (int64_t)c.n_kv_heads * c.head_dim;
  const int64_t Mx = (int64_t)c.max_batch * h->n_tok + ROW_PAD, Max = (int64_t)c.max_batch * c.horizon + ROW_PAD;
  std::vector<CUtensorMap> m(loop::MAP_LAYER0 + 4 * (size_t)c.n_layers);
  bool ok = tc::make_map_bf16(&m[loop::MAP_W2], h->W2, D, D, 128) &&
            tc::make_map_bf16(&m[loop::MAP_A_EZ], h->ez, Max, D, loop::TOK) &&
            tc::make_map_bf16(&m[loop::MAP_A_HB], h->hb, Mx, D, loop::TOK) &&
            tc::make_map_bf16(&m[loop::MAP_A_ATT], h->att, Mx, Q, loop::TOK) &&
            tc::make_map_bf16(&m[loop::MAP_A_MLP], h->mlp, Mx, F, loop::TOK) &&
            tc::make_map_bf16(&m[loop::MAP_KV2D], h->qkv, Mx, Q + 2 * KV, attn::KEY_BLOCK);
  m[loop::MAP_Q3D] = h->m_q;
  for (int l = 0; l < c.n_layers && ok; ++l) {
    LayerWeights& L = h->layers[l];
    ok = tc::make_map_bf16(&m[loop::MAP_LAYER0 + 4 * l + 0], L.wqkv, Q + 2 * KV, D, 128) &&
         tc::make_map_bf16(&m[loop::MAP_LAYER0 + 4 * l + 1], L.wo, D, Q, 128) &&
         tc::make_map_bf16(&m[loop::MAP_LAYER0 + 4 * l + 2], L.wgu, 2 * F, D, 128) &&
         tc::make_map_bf16(&m[loop::MAP_LAYER0 + 4 * l + 3], L.wd, D, F, 128);
  }
  if (!ok) return ADIT_E_CUDA;
  CU_TRY(h, cudaMemcpy(h->maps_dev, m.data(), m.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice));
  return ADIT_OK;
}

// One request's prefix cache as a 3-D tensor (channel, row, plane = (layer, K|V, kv head)) whose row extent is the
// request's prefix length: rows at or beyond it are never read, the copy engine writes zeros for them.
static bool make_map_prefix(CUtensorMap* m, const void* base, int dh, int plen, int p_cap, int64_t planes) {
  tc::EncodeTiledFn fn = tc::encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t gdim[3] = {(cuuint64_t)dh, (cuuint64_t)(plen > 0 ? plen : 1), (cuuint64_t)planes};
  cuuint64_t gstride[2] = {(cuuint64_t)dh * 2, (cuuint64_t)p_cap * dh * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)attn::KEY_BLOCK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int loop_clusters_for(const adit_handle* h, int sm_budget) {
  const int G = (sm_budget <= 0 || sm_budget >= h->sm_count) ? h->sm_count : sm_budget;
  int cl = G / loop::CS;
  return cl > h->loop_clusters ? h->loop_clusters : cl;
}
static bool loop_eligible(const adit_handle* h, int B, int sm_budget) {
  return h->loop_ok && B <= loop::MAXB && B * h->n_tok <= loop::TOK && loop_clusters_for(h, sm_budget) >= 1;
}

static int denoise_loop(adit_handle* h, int B, const PrefixTable& pt, const float* state, const float* noise, int K,
                        int sm_budget, cudaStream_t st, float* out) {
  const adit_config& c = h->cfg;
  const int D = c.d_model, A = c.action_dim, S = c.state_dim, Ta = c.horizon;
  const int clusters = loop_clusters_for(h, sm_budget);
  loop::LoopParams p{};
  const int64_t planes = (int64_t)c.n_layers * 2 * c.n_kv_heads;
  for (int b = 0; b < loop::MAXB; ++b) {
    p.plen[b] = b < B ? pt.len[b] : 0;
    if (b < B && pt.len[b] > 0) {
      if (!make_map_prefix(&p.pk[b], pt.kv[b], c.head_dim, pt.len[b], c.max_prefix_len, planes)) return ADIT_E_CUDA;
    } else {
      p.pk[b] = h->m_q;  // never used (no prefix block): any valid map
    }
  }
  p.maps = h->maps_dev;
  // (rows past the call's last token read as zeros: a masked key's V row must be finite for P V)
  if (!tc::make_map_bf16(&p.kv2d, h->qkv, (uint64_t)B * h->n_tok, (uint64_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim, attn::KEY_BLOCK))
    return ADIT_E_CUDA;
  for (int i = 0; i < loop::G_COUNT; ++i) p.g[i] = h->loop_g[i];
  p.L = c.n_layers; p.K = K; p.D = D; p.F = c.d_ff; p.n_q_heads = c.n_q_heads; p.n_kv_heads = c.n_kv_heads;
  p.n_tok = h->n_tok; p.horizon = Ta; p.A = A; p.B = B; p.M = B * h->n_tok; p.Ma = B * Ta;
  p.n_clusters = clusters;
  const int Gq = c.n_q_heads / c.n_kv_heads;
  p.n_row_tiles = (h->n_tok * Gq + 127) / 128;
  p.att_units = B * c.n_kv_heads * p.n_row_tiles;
  p.ssq_ld = c.max_batch * h->n_tok + ROW_PAD;
  p.n_dtiles = D / 128;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)c.head_dim);
  p.eps = c.rms_eps; p.dt = 1.0f / (float)K;
  p.x = h->x; p.h = h->h; p.ssq = h->ssq; p.out = out;
  p.hb = (bf16*)h->hb; p.qkv = (bf16*)h->qkv; p.att = (bf16*)h->att; p.mlp = (bf16*)h->mlp; p.ez = (bf16*)h->ez;
  p.Wfold = h->Wfold; p.bfold = h->bfold; p.ctime = h->ctime; p.hs = h->hs; p.ssq_state = h->rstd_state;
  p.Wout = h->Wout; p.bout = h->bout; p.b2 = h->b2; p.hsb = h->hsb;
  p.counters = h->loop_counters; p.status = h->status_dev; p.xscratch = h->loop_scratch;
  p.timeout_ns = h->wait_limit_ns; p.debug_skip_level = h->debug_skip_level;
  p.state_mask = (c.flags & ADIT_FLAG_STATE_BLOCK_MASK) ? 1 : 0;
  const int n_levels = K * (3 + 5 * c.n_layers), n_blocks = clusters * loop::CS;
  p.trace = nullptr;
  if (h->tracing) {
    const size_t need = (size_t)n_levels * n_blocks * 8;
    if (need > h->loop_trace_cap) {
      void* q = nullptr;
      CU_TRY(h, cudaMalloc(&q, need * 8));
      h->allocs.push_back(q);
      h->loop_trace = (unsigned long long*)q; h->loop_trace_cap = need;
    }
    CU_TRY(h, cudaMemsetAsync(h->loop_trace, 0, need * 8, st));
    p.trace = h->loop_trace;
    h->loop_trace_levels = n_levels; h->loop_trace_blocks = n_blocks; h->loop_trace_layers = c.n_layers;
  }
  const bool capturing = stream_is_capturing(st);  // (a captured call is ordered by the caller's graph, not by events here)
  if (!capturing) {
    // order this call behind loop kernels of other handles that it would not fit beside
    std::lock_guard<std::mutex> lock(g_loop_mutex);
    int busy = 0;
    for (auto it = g_loop_inflight.begin(); it != g_loop_inflight.end();) {
      if (it->h != h && it->device == h->device && cudaEventQuery(it->ev) == cudaSuccess) it = g_loop_inflight.erase(it);
      else { if (it->h != h && it->device == h->device) busy += it->clusters; ++it; }
    }
    cudaGetLastError();  // (cudaErrorNotReady from the queries is not an error)
    if (busy + clusters > h->loop_clusters)
      for (auto& e : g_loop_inflight)
        if (e.h != h && e.device == h->device) CU_TRY(h, cudaStreamWaitEvent(st, e.ev, 0));
  }
  {
    ProfScope ps(h, KC_PROLOGUE, st);
    int blocks = (p.Ma * A + 255) / 256;
    if (blocks < B) blocks = B;
    loop::loop_setup_kernel<<<blocks, 256, 0, st>>>(h->loop_counters, noise, state, h->x, p.Ma * A, h->Ws, h->bs, h->hs, h->hsb,
                                                   h->rstd_state, B, S, D);
    h->launches++;
  }
  {
    ProfScope ps(h, KC_LOOP, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_blocks);
    cfg.blockDim = dim3(loop::THREADS);
    cfg.dynamicSmemBytes = loop::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = loop::CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = h->use_pdl ? 2 : 1;
    cudaError_t e = c.head_dim == 64    ? cudaLaunchKernelEx(&cfg, loop::adit_loop_kernel<64>, p)
                    : c.head_dim == 128 ? cudaLaunchKernelEx(&cfg, loop::adit_loop_kernel<128>, p)
                                        : cudaLaunchKernelEx(&cfg, loop::adit_loop_kernel<256>, p);
    CU_TRY(h, e);
    h->launches++;
  }
  if (!capturing) {
    std::lock_guard<std::mutex> lock(g_loop_mutex);
    CU_TRY(h, cudaEventRecord(h->loop_ev, st));
    bool found = false;
    for (auto& e : g_loop_inflight)
      if (e.h == h) { e.clusters = clusters; found = true; }
    if (!found) g_loop_inflight.push_back({h, h->device, h->loop_ev, clusters});
  }
  return ADIT_OK;
}

// Tensor-core loop (bf16).  The per-call descriptor goes to the device through a one-block kernel; the
// rest of the call is one launch of a graph captured once per (B, K, budget) and cached in the handle.
static int denoise_tc(adit_handle* h, int B, const PrefixTable& pt, const float* state, const float* noise, int K,
                      int sm_budget, cudaStream_t st, float* out) {
  const adit_config& c = h->cfg;
  const int G = (sm_budget <= 0 || sm_budget >= h->sm_count) ? h->sm_count : sm_budget;
  if (stream_is_capturing(st)) {
    // Inside a caller's stream capture only pure enqueueing is possible: the time vectors for this K must exist
    // from an earlier call (they are computed by kernels that a graph replay must not repeat on other data).
    if (h->ctime_steps != K || h->profiling) return ADIT_E_UNSUPPORTED;
  }
  if (h->ctime_steps != K) {
    // c_k = tau(k/K) . W1[D:, :] + b1 depends on K only: computed when K changes and kept
    const int Tm = c.time_emb_dim, D = c.d_model;
    int n = K * (Tm / 2);
    ProfScope ps(h, KC_PROLOGUE, st);
    time_table_kernel<<<(n + 127) / 128, 128, 0, st>>>(h->tau, K, Tm, (double)c.t_min_period, (double)c.t_max_period);
    h->launches++;
    launch_ref_gemm<float, bf16, float, EPI_STORE_F32, false>(h, KC_PROLOGUE, st, h->tau, Tm, (const bf16*)h->W1t, Tm,
                                                              K, D, Tm, EpiArgs{h->ctime, D, nullptr, h->b1, 0});
    h->ctime_steps = K;
  }
  if (loop_eligible(h, B, sm_budget)) return denoise_loop(h, B, pt, state, noise, K, sm_budget, st, out);
  CallDesc d;
  d.pt = pt; d.state = state; d.noise = noise; d.out = out;
  set_desc_kernel<<<1, 32, 0, st>>>(d, h->desc_dev);
  h->launches++;
  if (!(c.flags & ADIT_FLAG_MMA_SYNC_ATTENTION)) {
    KvMaps km;
    const int64_t planes = (int64_t)c.n_layers * 2 * c.n_kv_heads;
    for (int b = 0; b < B; ++b) {
      if (pt.len[b] > 0) { if (!make_map_prefix(&km.pk[b], pt.kv[b], c.head_dim, pt.len[b], c.max_prefix_len, planes)) return ADIT_E_CUDA; }
      else km.pk[b] = h->m_sfx;  // never used (no prefix block): any valid map
    }
    set_kvmaps_kernel<<<1, 128, 0, st>>>(km, h->kvmaps_dev, B);
    h->launches++;
  }
  CU_TRY(h, cudaGetLastError());
  // (inside a caller's capture the kernels are recorded straight into the caller's graph)
  if (!h->use_graph || h->profiling || stream_is_capturing(st)) return enqueue_tc(h, B, K, G, st);

  auto key = std::make_tuple(B, K, G);
  auto it = h->graphs.find(key);
  if (it == h->graphs.end()) {
    const int64_t before = h->launches;
    cudaGraph_t graph = nullptr;
    CU_TRY(h, cudaStreamBeginCapture(h->cap_stream, cudaStreamCaptureModeThreadLocal));
    int rc = enqueue_tc(h, B, K, G, h->cap_stream);
    cudaError_t e = cudaStreamEndCapture(h->cap_stream, &graph);
    const int64_t n_launch = h->launches - before;
    h->launches = before;
    if (rc != ADIT_OK || e != cudaSuccess || !graph) {
      if (graph) cudaGraphDestroy(graph);
      if (e != cudaSuccess) h->last_cuda = (int)e;
      cudaGetLastError();
      return rc != ADIT_OK ? rc : ADIT_E_CUDA;
    }
    cudaGraphExec_t exec = nullptr;
    e = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    CU_TRY(h, e);
    it = h->graphs.emplace(key, adit_handle::GraphEntry{exec, n_launch}).first;
  }
  CU_TRY(h, cudaGraphLaunch(it->second.exec, st));
  h->launches += it->second.launches;
  return ADIT_OK;
}

static int validate_call(adit_handle* h, int B, const void* const* prefix_kv, const int32_t* prefix_len,
                         const float* state, const float* noise, int K, float* out, PrefixTable* pt) {
  if (!h || !prefix_kv || !prefix_len || !state || !noise || !out) return ADIT_E_INVALID;
  if (B < 1 || K < 1) return ADIT_E_INVALID;
  if (B > h->cfg.max_batch || K > ADIT_MAX_STEPS) return ADIT_E_CAPACITY;
  if (!h->loaded) return ADIT_E_NOT_LOADED;
  for (int b = 0; b < B; ++b) {
    if (prefix_len[b] < 0 || prefix_len[b] > h->cfg.max_prefix_len) return ADIT_E_INVALID;
    if (!prefix_kv[b] && h->cfg.max_prefix_len > 0) return ADIT_E_INVALID;
    if (((uintptr_t)prefix_kv[b]) & 15) return ADIT_E_INVALID;
    pt->kv[b] = prefix_kv[b];
    pt->len[b] = prefix_len[b];
  }
  for (int b = B; b < 64; ++b) { pt->kv[b] = nullptr; pt->len[b] = 0; }
  if ((((uintptr_t)state) & 3) || (((uintptr_t)noise) & 3) || (((uintptr_t)out) & 3)) return ADIT_E_INVALID;
  return ADIT_OK;
}

static int denoise_dispatch(adit_handle* h, int B, const PrefixTable& pt, const float* state, const float* noise,
                            int K, int sm_budget, cudaStream_t st, float* out) {
  if (h->cfg.dtype == ADIT_DTYPE_FP32) return denoise_reference<float>(h, B, pt, state, noise, K, st, out);
  if (use_reference_kernels(h->cfg)) return denoise_reference<bf16>(h, B, pt, state, noise, K, st, out);
  return denoise_tc(h, B, pt, state, noise, K, sm_budget, st, out);
}

extern "C" int adit_denoise(adit_handle* h, int B, const void* const* prefix_kv, const int32_t* prefix_len,
                            const float* state, const float* noise, int K, int sm_budget, void* stream,
                            float* out_actions) {
  PrefixTable pt;
  int rc = validate_call(h, B, prefix_kv, prefix_len, state, noise, K, out_actions, &pt);
  if (rc) return rc;
  CU_TRY(h, cudaSetDevice(h->device));
  return denoise_dispatch(h, B, pt, state, noise, K, sm_budget, (cudaStream_t)stream, out_actions);
}

extern "C" int adit_denoise_host(adit_handle* h, int B, const void* const* prefix_kv, const int32_t* prefix_len,
                                 const float* state_host, const float* noise_host, int K, int sm_budget, void* stream,
                                 float* out_actions_host) {
  PrefixTable pt;
  int rc = validate_call(h, B, prefix_kv, prefix_len, state_host, noise_host, K, out_actions_host, &pt);
  if (rc) return rc;
  CU_TRY(h, cudaSetDevice(h->device));
  cudaStream_t st = (cudaStream_t)stream;
  const adit_config& c = h->cfg;
  size_t nb_state = (size_t)B * c.state_dim * 4, nb_x = (size_t)B * c.horizon * c.action_dim * 4;
  CU_TRY(h, cudaMemcpyAsync(h->state_dev, state_host, nb_state, cudaMemcpyHostToDevice, st));
  CU_TRY(h, cudaMemcpyAsync(h->noise_dev, noise_host, nb_x, cudaMemcpyHostToDevice, st));
  rc = denoise_dispatch(h, B, pt, h->state_dev, h->noise_dev, K, sm_budget, st, h->noise_dev);
  if (rc) return rc;
  CU_TRY(h, cudaMemcpyAsync(out_actions_host, h->noise_dev, nb_x, cudaMemcpyDeviceToHost, st));
  CU_TRY(h, cudaStreamSynchronize(st));
  return ADIT_OK;
}

extern "C" const char* adit_profile_class_name(int cls) {
  static const char* names[KC_COUNT] = {"prologue", "embed", "norm", "gemm_qkv", "attention", "gemm_o",
                                        "gemm_gateup", "gemm_down", "final", "reduce", "loop"};
  return (cls >= 0 && cls < KC_COUNT) ? names[cls] : "";
}

extern "C" int adit_profile_enable(adit_handle* h, int on) {
  if (!h) return ADIT_E_INVALID;
  h->profiling = on != 0;
  return ADIT_OK;
}

extern "C" int adit_profile_read(adit_handle* h, double* total_ms, int64_t* launches) {
  if (!h || !total_ms || !launches) return ADIT_E_INVALID;
  CU_TRY(h, cudaSetDevice(h->device));
  CU_TRY(h, cudaDeviceSynchronize());
  for (int i = 0; i < KC_COUNT; ++i) { total_ms[i] = 0.0; launches[i] = 0; }
  for (auto& r : h->prof) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) { total_ms[r.cls] += ms; launches[r.cls]++; }
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  h->prof.clear();
  return ADIT_OK;
}

extern "C" int adit_trace_enable(adit_handle* h, int on) {
  if (!h) return ADIT_E_INVALID;
  CU_TRY(h, cudaSetDevice(h->device));
  CU_TRY(h, cudaDeviceSynchronize());
  if (on && !h->trace_dev) {
    h->trace_cap = (size_t)1 << 21;  // 16 MB of timestamps
    CU_TRY(h, cudaMalloc((void**)&h->trace_dev, h->trace_cap * 8));
    h->allocs.push_back(h->trace_dev);
  }
  h->tracing = on != 0;
  // launch graphs recorded so far carry the old setting: drop them
  for (auto& g : h->graphs) cudaGraphExecDestroy(g.second.exec);
  h->graphs.clear();
  return ADIT_OK;
}

extern "C" int64_t adit_trace_read(adit_handle* h, int64_t* records, int64_t max_records) {
  if (!h || !records || max_records < 0) return ADIT_E_INVALID;
  if (!h->trace_dev) return 0;
  CU_TRY(h, cudaSetDevice(h->device));
  CU_TRY(h, cudaDeviceSynchronize());
  std::vector<unsigned long long> buf(h->trace_off);
  if (h->trace_off) CU_TRY(h, cudaMemcpy(buf.data(), h->trace_dev, h->trace_off * 8, cudaMemcpyDeviceToHost));
  int64_t n = 0;
  for (const auto& r : h->trace_recs) {
    if (n >= max_records) break;
    unsigned long long s_min = ~0ull, s_max = 0, e_min = ~0ull, e_max = 0, w_min = ~0ull, w_max = 0, m_min = ~0ull, m_max = 0;
    for (int b = 0; b < r.grid; ++b) {
      unsigned long long s = buf[r.off + 4 * b], w = buf[r.off + 4 * b + 1], e = buf[r.off + 4 * b + 2];
      unsigned long long m = buf[r.off + 4 * b + 3];
      if (m && m < m_min) m_min = m;
      if (m > m_max) m_max = m;
      if (s < s_min) s_min = s;
      if (s > s_max) s_max = s;
      if (e < e_min) e_min = e;
      if (e > e_max) e_max = e;
      if (w && w < w_min) w_min = w;
      if (w > w_max) w_max = w;
    }
    int64_t* o = records + n * 10;
    o[0] = r.cls; o[1] = r.grid; o[2] = (int64_t)s_min; o[3] = (int64_t)s_max; o[4] = (int64_t)e_min; o[5] = (int64_t)e_max;
    o[6] = w_max ? (int64_t)w_min : 0; o[7] = (int64_t)w_max;
    o[8] = m_max ? (int64_t)m_min : 0; o[9] = (int64_t)m_max;
    ++n;
  }
  return n;
}


extern "C" int adit_clear_status(adit_handle* h) {
  if (!h) return ADIT_E_INVALID;
  CU_TRY(h, cudaSetDevice(h->device));
  CU_TRY(h, cudaDeviceSynchronize());
  *h->status_host = 0;
  return ADIT_OK;
}

extern "C" int adit_debug_wait_limit(adit_handle* h, int limit_ms, int withhold_level) {
  if (!h || limit_ms < 1 || withhold_level < -1 || withhold_level >= loop::LV_COUNT) return ADIT_E_INVALID;
  h->wait_limit_ns = (unsigned long long)limit_ms * 1000000ull;
  h->debug_skip_level = withhold_level;
  return ADIT_OK;
}

extern "C" int adit_uses_persistent_loop(adit_handle* h, int B, int sm_budget) {
  if (!h || B < 1) return ADIT_E_INVALID;
  if (h->cfg.dtype != ADIT_DTYPE_BF16 || use_reference_kernels(h->cfg)) return 0;
  return loop_eligible(h, B, sm_budget) ? loop_clusters_for(h, sm_budget) * loop::CS : 0;
}

extern "C" int64_t adit_loop_trace_read(adit_handle* h, int64_t* records, int64_t max_records) {
  if (!h || !records || max_records < 0) return ADIT_E_INVALID;
  if (!h->loop_trace || !h->loop_trace_levels) return 0;
  CU_TRY(h, cudaSetDevice(h->device));
  CU_TRY(h, cudaDeviceSynchronize());
  const int nl = h->loop_trace_levels, nb = h->loop_trace_blocks, per_step = 3 + 5 * h->loop_trace_layers;
  std::vector<unsigned long long> buf((size_t)nl * nb * 8);
  CU_TRY(h, cudaMemcpy(buf.data(), h->loop_trace, buf.size() * 8, cudaMemcpyDeviceToHost));
  int64_t n = 0;
  for (int lv = 0; lv < nl && n < max_records; ++lv, ++n) {
    const int j = lv % per_step;
    const int type = j == 0 ? loop::LV_EMBED_IN : j == 1 ? loop::LV_W2 : j == per_step - 1 ? loop::LV_FINAL : loop::LV_QKV + (j - 2) % 5;
    unsigned long long s_min = ~0ull, mx[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int blocks = 0;
    for (int b = 0; b < nb; ++b) {
      const unsigned long long* t = &buf[((size_t)lv * nb + b) * 8];
      if (!t[0]) continue;
      ++blocks;
      if (t[0] < s_min) s_min = t[0];
      for (int k = 0; k < 8; ++k)
        if (t[k] > mx[k]) mx[k] = t[k];
    }
    int64_t* o = records + n * 11;
    o[0] = type; o[1] = blocks; o[2] = blocks ? (int64_t)s_min : 0;
    for (int k = 0; k < 8; ++k) o[3 + k] = (int64_t)mx[k];
  }
  return n;
}

extern "C" int64_t adit_debug_copy(adit_handle* h, const char* name, void* host_dst, size_t nbytes) {
  if (!h || !name || !host_dst) return ADIT_E_INVALID;
  const adit_config& c = h->cfg;
  const int64_t Mx = (int64_t)c.max_batch * h->n_tok, Ma = (int64_t)c.max_batch * c.horizon;
  const int64_t Q = (int64_t)c.n_q_heads * c.head_dim, KV = (int64_t)c.n_kv_heads * c.head_dim;
  const void* src = nullptr;
  size_t size = 0;
  std::string n(name);
  if (n == "x") { src = h->x; size = Ma * c.action_dim * 4; }
  else if (n == "h") { src = h->h; size = Mx * c.d_model * 4; }
  else if (n == "rstd") { src = h->rstd; size = Mx * 4; }
  else if (n == "ctime") { src = h->ctime; size = (size_t)ADIT_MAX_STEPS * c.d_model * 4; }
  else if (n == "qkv") { src = h->qkv; size = Mx * (Q + 2 * KV) * h->esz; }
  else if (n == "att") { src = h->att; size = Mx * Q * h->esz; }
  else if (n == "mlp") { src = h->mlp; size = Mx * c.d_ff * h->esz; }
  else if (n == "hb") { src = h->hb; size = Mx * c.d_model * h->esz; }
  else return ADIT_E_INVALID;
  if (nbytes < size) size = nbytes;
  CU_TRY(h, cudaSetDevice(h->device));
  CU_TRY(h, cudaDeviceSynchronize());
  CU_TRY(h, cudaMemcpy(host_dst, src, size, cudaMemcpyDeviceToHost));
  return (int64_t)size;
}

// ---------------------------------------------------------------------------------------------
// A stream confined to an SM partition by the driver (green context): the paper's own way of restricting the VLM stage
// ---------------------------------------------------------------------------------------------
struct adit_green_stream {
  int device;
  CUgreenCtx ctx;
  CUstream stream;
  int sm_count;
};

template <typename F>
static F driver_fn(const char* name) {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) return nullptr;
  return (F)p;
}

extern "C" int adit_green_stream_create(int device, int sm_count, adit_green_stream** out) {
  if (!out || sm_count < 1) return ADIT_E_INVALID;
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  if (cudaFree(0) != cudaSuccess) return ADIT_E_CUDA;  // (the primary context exists)
  auto get_res = driver_fn<CUresult (*)(CUdevice, CUdevResource*, CUdevResourceType)>("cuDeviceGetDevResource");
  auto split = driver_fn<CUresult (*)(CUdevResource*, unsigned int*, const CUdevResource*, CUdevResource*, unsigned int, unsigned int)>(
      "cuDevSmResourceSplitByCount");
  auto gen_desc = driver_fn<CUresult (*)(CUdevResourceDesc*, CUdevResource*, unsigned int)>("cuDevResourceGenerateDesc");
  auto ctx_create = driver_fn<CUresult (*)(CUgreenCtx*, CUdevResourceDesc, CUdevice, unsigned int)>("cuGreenCtxCreate");
  auto ctx_destroy = driver_fn<CUresult (*)(CUgreenCtx)>("cuGreenCtxDestroy");
  auto stream_create = driver_fn<CUresult (*)(CUstream*, CUgreenCtx, unsigned int, int)>("cuGreenCtxStreamCreate");
  auto dev_get = driver_fn<CUresult (*)(CUdevice*, int)>("cuDeviceGet");
  if (!get_res || !split || !gen_desc || !ctx_create || !ctx_destroy || !stream_create || !dev_get) return ADIT_E_UNSUPPORTED;
  CUdevice dev;
  if (dev_get(&dev, device) != CUDA_SUCCESS) return ADIT_E_CUDA;
  CUdevResource all, part, rest;
  if (get_res(dev, &all, CU_DEV_RESOURCE_TYPE_SM) != CUDA_SUCCESS) return ADIT_E_UNSUPPORTED;
  if ((unsigned)sm_count > all.sm.smCount) return ADIT_E_CAPACITY;
  unsigned int groups = 1;
  // one group of at least sm_count SMs (the driver rounds up to its granularity); the remainder is not used here
  if (split(&part, &groups, &all, &rest, 0, (unsigned)sm_count) != CUDA_SUCCESS || groups != 1) return ADIT_E_UNSUPPORTED;
  CUdevResourceDesc desc;
  if (gen_desc(&desc, &part, 1) != CUDA_SUCCESS) return ADIT_E_CUDA;
  adit_green_stream* g = new (std::nothrow) adit_green_stream();
  if (!g) return ADIT_E_INVALID;
  g->device = device; g->sm_count = (int)part.sm.smCount; g->stream = nullptr;
  if (ctx_create(&g->ctx, desc, dev, CU_GREEN_CTX_DEFAULT_STREAM) != CUDA_SUCCESS) { delete g; return ADIT_E_CUDA; }
  if (stream_create(&g->stream, g->ctx, CU_STREAM_NON_BLOCKING, 0) != CUDA_SUCCESS) { ctx_destroy(g->ctx); delete g; return ADIT_E_CUDA; }
  *out = g;
  return ADIT_OK;
}
extern "C" void* adit_green_stream_handle(adit_green_stream* g) { return g ? (void*)g->stream : nullptr; }
extern "C" int adit_green_stream_sm_count(adit_green_stream* g) { return g ? g->sm_count : 0; }
extern "C" int adit_green_stream_destroy(adit_green_stream* g) {
  if (!g) return ADIT_OK;
  cudaSetDevice(g->device);
  if (g->stream) { cudaStreamSynchronize((cudaStream_t)g->stream); cudaStreamDestroy((cudaStream_t)g->stream); }
  auto ctx_destroy = driver_fn<CUresult (*)(CUgreenCtx)>("cuGreenCtxDestroy");
  if (ctx_destroy) ctx_destroy(g->ctx);
  delete g;
  return ADIT_OK;
}

// Test and measurement aids (stand-alone attention and projection entry points, phase stamps, the streaming-read
// probe, the stand-in GEMM of the VLM stage): in a file of their own, and left out of the build with -DADIT_NO_AIDS.
#ifndef ADIT_NO_AIDS
#include "adit_aids.cuh"
#endif
