// Test and measurement aids of the ADiT library, included at the end of adit_api.cu (one translation unit: they launch
// the same kernels through the same host helpers, and a second unit would instantiate every kernel twice):
// the stand-alone ragged-prefix attention (allocating and allocation-free entry points), the stand-alone projection with
// its phase stamps, the planner query, the streaming-read probe and the looping stand-in GEMM of the VLM stage.
// None of it is on the path of adit_denoise; -DADIT_NO_AIDS builds the library without it.
#pragma once

// ---------------------------------------------------------------------------------------------
// Stand-alone ragged-prefix attention (test aid): the kernels of the loop on caller-supplied buffers.
// ---------------------------------------------------------------------------------------------
// Phase-stamp buffer of adit_debug_gemm_stamps: [1024 blocks][16] uint64 on the device it was armed on.  The
// attention kernel's per-key-block log of block 0 starts at element 8192, so attention grids may use 512 blocks.
static unsigned long long* g_gemm_dbg = nullptr;
static int g_gemm_dbg_device = -1;
extern "C" int adit_debug_stamps_selected(int armed_device, int device, int grid_blocks, int is_attention) {
  if (armed_device < 0 || armed_device != device || grid_blocks < 1) return 0;
  return grid_blocks <= (is_attention ? 512 : 1024) ? 1 : 0;
}
static unsigned long long* stamp_buffer_for(int grid_blocks, bool is_attention) {
  int dev = -1;
  if (!g_gemm_dbg || cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  return adit_debug_stamps_selected(g_gemm_dbg_device, dev, grid_blocks, is_attention ? 1 : 0) ? g_gemm_dbg : nullptr;
}
__global__ void set_table_kernel(PrefixTable t, PrefixTable* __restrict__ dst, int* __restrict__ status) {
  if (threadIdx.x == 0) { *dst = t; if (status) *status = 0; }
}

struct AttnProblem {
  int B, n_tokens, n_q_heads, n_kv_heads, head_dim, p_cap, layer, splits;
};

static int validate_attention(const AttnProblem& q, const void* qkv, const void* const* prefix_kv,
                              const int32_t* prefix_len, const void* out_att, PrefixTable* pt) {
  if (!qkv || !prefix_kv || !prefix_len || !out_att) return ADIT_E_INVALID;
  if ((((uintptr_t)qkv) & 15) || (((uintptr_t)out_att) & 15)) return ADIT_E_INVALID;  // 16-byte copies and stores
  if (q.B < 1 || q.n_tokens < 1 || q.n_q_heads < 1 || q.n_kv_heads < 1 || q.p_cap < 0 || q.layer < 0) return ADIT_E_INVALID;
  if (q.n_q_heads % q.n_kv_heads) return ADIT_E_INVALID;
  if (q.B > ADIT_MAX_BATCH) return ADIT_E_CAPACITY;
  if (q.head_dim != 64 && q.head_dim != 128 && q.head_dim != 256) return ADIT_E_UNSUPPORTED;
  if (q.splits < 1 || q.splits > 32) return ADIT_E_INVALID;
  for (int b = 0; b < q.B; ++b) {
    if (prefix_len[b] < 0 || prefix_len[b] > q.p_cap) return ADIT_E_INVALID;
    if ((!prefix_kv[b] && q.p_cap > 0) || (((uintptr_t)prefix_kv[b]) & 15)) return ADIT_E_INVALID;
    pt->kv[b] = prefix_kv[b];
    pt->len[b] = prefix_len[b];
  }
  for (int b = q.B; b < 64; ++b) { pt->kv[b] = nullptr; pt->len[b] = 0; }
  return ADIT_OK;
}

static size_t attention_scratch_bytes(const AttnProblem& q) {
  const size_t rows = (size_t)q.splits * q.B * q.n_tokens * q.n_q_heads;
  return q.splits > 1 ? rows * q.head_dim * 4 + rows * 2 * 4 : 0;
}

template <int DH>
static cudaError_t attention_launch_dh(const attn::AttnArgs& a, int nw, int grid, int merge_grid, int64_t n_qrows,
                                       const PrefixTable* pt_dev, cudaStream_t st) {
  (void)nw;
  CUtensorMap mq, msfx;
  if (!tc::make_map_bf16(&msfx, a.qkv, (uint64_t)a.batch * a.n_tokens, (uint64_t)a.ldqkv, attn::KEY_BLOCK)) return cudaErrorInvalidValue;
  attn::AttnArgs b = a;
  b.q_tma = tc::make_map_q(&mq, a.qkv, (uint64_t)a.batch * a.n_tokens, (uint64_t)a.ldqkv, DH, (uint32_t)a.n_q_heads,
                           (uint32_t)(a.n_q_heads / a.n_kv_heads)) ? 1 : 0;
  if (!b.q_tma) memset(&mq, 0, sizeof(mq));
  auto kern = pick_attn_kernel<DH>(b.dbg != nullptr, b.splits > 1, b.q_tma != 0);
  kern<<<grid, attn::TC_THREADS, attn::attn_tc_smem_bytes<DH>(), st>>>(mq, msfx, b, pt_dev);
  if (a.splits > 1)
    (a.splits > 4 ? attn::attn_merge_kernel<DH, bf16, 16, (DH >= 128 ? 2 : 1)> : attn::attn_merge_kernel<DH, bf16, 4>)
        <<<a.splits > 4 ? merge_grid * (DH >= 128 ? 2 : 1) : merge_grid, 128, 0, st>>>(
        (const bf16*)a.part_o, a.part_ml, a.splits, n_qrows, a.n_q_heads, a.att, a.ldatt, nullptr);
  return cudaGetLastError();
}

// Enqueue attention on `st`.  `scratch` holds the key-split partials (attention_scratch_bytes) and
// `pt_dev` the device copy of the prefix table (written here by a small kernel).
static cudaError_t attention_enqueue(const AttnProblem& q, const PrefixTable& pt, const void* qkv, void* out_att,
                                     unsigned char* scratch, PrefixTable* pt_dev, int* status_dev, KvMaps* maps_dev,
                                     cudaStream_t st) {
  const int G = q.n_q_heads / q.n_kv_heads, R = q.n_tokens * G;
  const int nw = R <= 32 ? 2 : 4;
  const int Q = q.n_q_heads * q.head_dim;
  attn::AttnArgs a{};
  a.qkv = (const bf16*)qkv; a.ldqkv = Q + 2 * q.n_kv_heads * q.head_dim; a.att = (bf16*)out_att; a.ldatt = Q;
  a.layer = q.layer; a.n_tokens = q.n_tokens; a.n_q_heads = q.n_q_heads; a.n_kv_heads = q.n_kv_heads;
  a.p_cap = q.p_cap; a.batch = q.B; a.n_row_tiles = (R + attn::TC_ROWS - 1) / attn::TC_ROWS; a.splits = q.splits;
  a.scale_log2 = 1.4426950408889634f / sqrtf((float)q.head_dim);
  const size_t rows = (size_t)q.splits * q.B * q.n_tokens * q.n_q_heads;
  a.part_o = scratch;
  a.dbg = stamp_buffer_for(q.B * q.n_kv_heads * ((R + attn::TC_ROWS - 1) / attn::TC_ROWS) * q.splits, true);
  a.part_ml = (float*)(scratch + rows * q.head_dim * 4);  // (the bf16 partials use half of the first region)
  a.status = status_dev;  // cleared by the table kernel, set to ADIT_E_TIMEOUT by a wait that runs out
  set_table_kernel<<<1, 32, 0, st>>>(pt, pt_dev, status_dev);
  {
    KvMaps km;
    const int64_t planes = (int64_t)(q.layer + 1) * 2 * q.n_kv_heads;   // the cache is indexed up to `layer`
    CUtensorMap any;
    if (!tc::make_map_bf16(&any, qkv, (uint64_t)q.B * q.n_tokens, (uint64_t)(Q + 2 * q.n_kv_heads * q.head_dim), attn::KEY_BLOCK))
      return cudaErrorInvalidValue;
    for (int b = 0; b < q.B; ++b) {
      if (pt.len[b] > 0) { if (!make_map_prefix(&km.pk[b], pt.kv[b], q.head_dim, pt.len[b], q.p_cap, planes)) return cudaErrorInvalidValue; }
      else km.pk[b] = any;
    }
    set_kvmaps_kernel<<<1, 128, 0, st>>>(km, maps_dev, q.B);
    a.kv_maps = maps_dev->pk;
  }
  const int grid = q.B * q.n_kv_heads * a.n_row_tiles * q.splits;
  const int64_t n_qrows = (int64_t)q.B * q.n_tokens * q.n_q_heads;
  const int mg = (int)((n_qrows + 3) / 4);
  if (q.head_dim == 64) return attention_launch_dh<64>(a, nw, grid, mg, n_qrows, pt_dev, st);
  if (q.head_dim == 128) return attention_launch_dh<128>(a, nw, grid, mg, n_qrows, pt_dev, st);
  return attention_launch_dh<256>(a, nw, grid, mg, n_qrows, pt_dev, st);
}

extern "C" int adit_debug_attention(int device, int B, int n_tokens, int n_q_heads, int n_kv_heads, int head_dim,
                                    int p_cap, int layer, const void* qkv, const void* const* prefix_kv,
                                    const int32_t* prefix_len, int splits, void* out_att, void* stream) {
  AttnProblem q{B, n_tokens, n_q_heads, n_kv_heads, head_dim, p_cap, layer, splits};
  PrefixTable pt;
  int rc = validate_attention(q, qkv, prefix_kv, prefix_len, out_att, &pt);
  if (rc) return rc;
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  if (init_attention_attrs() != cudaSuccess) return ADIT_E_CUDA;
  unsigned char* scratch = nullptr;
  PrefixTable* pt_dev = nullptr;
  const size_t nb = attention_scratch_bytes(q);
  const size_t maps_off = (sizeof(PrefixTable) + 16 + 255) / 256 * 256;
  if (cudaMalloc((void**)&pt_dev, maps_off + sizeof(KvMaps)) != cudaSuccess) return ADIT_E_CUDA;
  if (nb && cudaMalloc((void**)&scratch, nb) != cudaSuccess) { cudaFree(pt_dev); return ADIT_E_CUDA; }
  cudaStream_t st = (cudaStream_t)stream;
  int* status_dev = (int*)((unsigned char*)pt_dev + sizeof(PrefixTable));
  cudaError_t e = attention_enqueue(q, pt, qkv, out_att, scratch, pt_dev, status_dev, (KvMaps*)((unsigned char*)pt_dev + maps_off), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  int hs = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&hs, status_dev, 4, cudaMemcpyDeviceToHost);
  cudaFree(pt_dev);
  if (scratch) cudaFree(scratch);
  if (e != cudaSuccess) return ADIT_E_CUDA;
  return hs ? ADIT_E_TIMEOUT : ADIT_OK;
}

// ---------------------------------------------------------------------------------------------
// adit_attention_static: the same attention, for callers that must not allocate device memory.
// Scratch (key-split partials + the device copy of the prefix table) lives in a fixed array that every
// GPU loading this library holds until the process exits.
// ---------------------------------------------------------------------------------------------
// [key-split partials | prefix table, status word (within 1 KB) | the call's prefix-cache tensor maps]
static __device__ __align__(256) unsigned char g_static_scratch[ADIT_STATIC_SCRATCH_BYTES + 1024 + sizeof(KvMaps)];
static_assert(sizeof(PrefixTable) + 16 <= 1024, "table and status word must fit their slot");
static unsigned char* g_static_scratch_addr[64] = {};  // device address of the array, per device ordinal

extern "C" int adit_attention_static(int device, int B, int n_tokens, int n_q_heads, int n_kv_heads, int head_dim,
                                     int p_cap, int layer, const void* qkv, const void* const* prefix_kv,
                                     const int32_t* prefix_len, int splits, void* out_att, void* stream) {
  AttnProblem q{B, n_tokens, n_q_heads, n_kv_heads, head_dim, p_cap, layer, splits};
  PrefixTable pt;
  int rc = validate_attention(q, qkv, prefix_kv, prefix_len, out_att, &pt);
  if (rc) return rc;
  if (attention_scratch_bytes(q) > ADIT_STATIC_SCRATCH_BYTES) return ADIT_E_CAPACITY;  // partials do not fit the fixed array
  if (device < 0 || device >= 64) return ADIT_E_INVALID;
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  if (!g_static_scratch_addr[device]) {
    // First call on this device: the array's name is only a host-side handle, the kernels need the
    // device address.  Looked up once per device, with that device current.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ADIT_E_CUDA;
    if (init_attention_attrs() != cudaSuccess) return ADIT_E_CUDA;
    g_static_scratch_addr[device] = (unsigned char*)p;
  }
  unsigned char* base = g_static_scratch_addr[device];
  PrefixTable* pt_dev = (PrefixTable*)(base + ADIT_STATIC_SCRATCH_BYTES);  // 256-byte aligned: the array is, and so is its size
  // Nothing in the scratch has to start at zero: every (split, row) partial that the merge reads is
  // written by the attention kernel of the same call, empty splits included.
  int* status_dev = (int*)(base + ADIT_STATIC_SCRATCH_BYTES + sizeof(PrefixTable));  // inside the array's last 256 bytes
  cudaError_t e = attention_enqueue(q, pt, qkv, out_att, base, pt_dev, status_dev, (KvMaps*)(base + ADIT_STATIC_SCRATCH_BYTES + 1024),
                                    (cudaStream_t)stream);
  return e == cudaSuccess ? ADIT_OK : ADIT_E_CUDA;
}

extern "C" int adit_attention_static_status(int device) {
  if (device < 0 || device >= 64) return ADIT_E_INVALID;
  if (!g_static_scratch_addr[device]) return ADIT_OK;  // never used on this device
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  int hs = 0;
  if (cudaMemcpy(&hs, g_static_scratch_addr[device] + ADIT_STATIC_SCRATCH_BYTES + sizeof(PrefixTable), 4, cudaMemcpyDeviceToHost) != cudaSuccess)
    return ADIT_E_CUDA;
  return hs ? ADIT_E_TIMEOUT : ADIT_OK;
}

extern "C" int adit_debug_plan(int n_tok, int n_feat, int k, int dual, int sm_count, int32_t* out) {
  if (!out || n_tok < 1 || n_feat < 1 || k < 64 || (k % 64) || sm_count < 1) return ADIT_E_INVALID;
  const tc::GemmPlan p = tc::plan_gemm(n_tok, n_feat, k, dual != 0, sm_count, true);
  out[0] = p.tile_tok; out[1] = p.n_ttiles; out[2] = p.n_ftiles; out[3] = p.splits; out[4] = p.stages; out[5] = p.kb_total;
  out[6] = p.acc_bufs; out[7] = p.issuers; out[8] = (int32_t)p.tmem_cols; out[9] = (int32_t)p.smem_bytes;
  out[10] = (int32_t)p.ring_bytes; out[11] = (int32_t)(p.est_us * 1000.0);
  return ADIT_OK;
}

extern "C" int adit_debug_plan_projection(int n_tok, int n_feat, int k, int dual, int sm_count, int allow_pair, int32_t* out) {
  if (!out || n_tok < 1 || n_feat < 1 || k < 64 || (k % 64) || sm_count < 1) return ADIT_E_INVALID;
  const tc::GemmPlan p = tc::plan_projection(n_tok, n_feat, k, dual != 0, sm_count, allow_pair != 0);
  out[0] = p.tile_tok; out[1] = p.n_ttiles; out[2] = p.n_ftiles; out[3] = p.splits; out[4] = p.stages; out[5] = p.kb_total;
  out[6] = p.acc_bufs; out[7] = p.issuers; out[8] = (int32_t)p.tmem_cols; out[9] = (int32_t)p.smem_bytes;
  out[10] = (int32_t)p.ring_bytes; out[11] = (int32_t)(p.est_us * 1000.0); out[12] = p.pair ? 1 : 0;
  return ADIT_OK;
}

extern "C" int adit_debug_gemm_stamps(unsigned long long* host_dst, int n_blocks) {
  if (!host_dst && n_blocks < 0) {  // disarm
    if (g_gemm_dbg) { cudaSetDevice(g_gemm_dbg_device); cudaDeviceSynchronize(); cudaFree(g_gemm_dbg); }
    g_gemm_dbg = nullptr; g_gemm_dbg_device = -1;
    return ADIT_OK;
  }
  if (!host_dst) {  // arm: allocate the stamp buffer on the current device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ADIT_E_CUDA;
    if (g_gemm_dbg && dev != g_gemm_dbg_device) return ADIT_E_INVALID;  // armed elsewhere: disarm first
    if (!g_gemm_dbg && cudaMalloc((void**)&g_gemm_dbg, 1024 * 16 * 8) != cudaSuccess) return ADIT_E_CUDA;
    g_gemm_dbg_device = dev;
    cudaMemset(g_gemm_dbg, 0, 1024 * 16 * 8);
    return ADIT_OK;
  }
  if (!g_gemm_dbg || n_blocks > 1024) return ADIT_E_INVALID;
  return cudaMemcpy(host_dst, g_gemm_dbg, (size_t)n_blocks * 128, cudaMemcpyDeviceToHost) == cudaSuccess ? ADIT_OK : ADIT_E_CUDA;
}

extern "C" int adit_debug_gemm(int device, int n_tok, int n_feat, int k, const void* a_bf16, const void* w_bf16,
                               float* out_f32, int splits, int sm_budget, void* stream) {
  if (!a_bf16 || !w_bf16 || !out_f32 || n_tok < 1 || n_feat < 1 || k < 64 || (k % 64)) return ADIT_E_INVALID;
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return ADIT_E_CUDA;
  if (prop.major != 10) return ADIT_E_UNSUPPORTED;
  if (tc::ensure_smem_attr() != cudaSuccess) return ADIT_E_CUDA;
  const int SM = prop.multiProcessorCount;
  if (splits == -2 && SM < 2) return ADIT_E_UNSUPPORTED;
  tc::GemmPlan p = splits == -2 ? tc::plan_gemm_pair(n_tok, n_feat, k, false, SM) : tc::plan_gemm(n_tok, n_feat, k, false, SM, true, splits % 100, splits / 100);
  CUtensorMap mw, ma;
  if (!tc::make_map_bf16(&mw, w_bf16, n_feat, k, tc::TILE_F) || !tc::make_map_bf16(&ma, a_bf16, n_tok, k, tc::token_box_rows(p)))
    return ADIT_E_CUDA;
  int* status = nullptr;
  float* tmp = nullptr;  // the kernel stores whole token tiles: give it the padding rows the library's buffers have
  const size_t rows_padded = (size_t)p.n_ttiles * p.tile_tok;
  if (cudaMalloc((void**)&status, 4) != cudaSuccess) return ADIT_E_CUDA;
  if (cudaMalloc((void**)&tmp, rows_padded * n_feat * 4) != cudaSuccess) { cudaFree(status); return ADIT_E_CUDA; }
  cudaMemset(status, 0, 4);
  cudaStream_t st = (cudaStream_t)stream;
  tc::GemmArgs g{};
  g.n_feat = n_feat; g.n_tok = n_tok; g.epi = EPI_STORE_F32; g.out = tmp; g.ldo = n_feat; g.status = status;
  const int G = (sm_budget <= 0 || sm_budget >= SM) ? SM : sm_budget;
  g.dbg = stamp_buffer_for(tc::gemm_grid(p, G), false);
  cudaError_t e = tc::launch_gemm(mw, ma, p, false, g, G, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(out_f32, tmp, (size_t)n_tok * n_feat * 4, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  int hs = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&hs, status, 4, cudaMemcpyDeviceToHost);
  cudaFree(status);
  cudaFree(tmp);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return ADIT_E_CUDA;
  }
  return hs ? hs : ((p.pair ? 9 : p.splits) * 1000000 + p.tile_tok * 1000 + p.stages);  // plan, for the test's information (9 = two-SM kernel)
}


// Makes a bounded device-side wait of the projection kernel run out, once, on purpose-built operands: block 0 of a
// small product (51 tokens x 2560 features x 1024, no k-split: no cluster is involved) never gets the tokens of its
// third k-block, so its issuing thread's wait on that stage expires after the kernel's two-second limit, the block
// records ADIT_E_TIMEOUT, lets its copies land, frees its tensor memory and returns like the others.  The same
// product is then run again untouched.  *first_status receives the status word after the first run (ADIT_E_TIMEOUT
// expected), the return value is the status after the second (ADIT_OK expected) or a host-side error.
extern "C" int adit_debug_gemm_timeout(int device, int* first_status, void* stream) {
  if (!first_status) return ADIT_E_INVALID;
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return ADIT_E_CUDA;
  if (prop.major != 10) return ADIT_E_UNSUPPORTED;
  if (tc::ensure_smem_attr() != cudaSuccess) return ADIT_E_CUDA;
  const int n_tok = 51, n_feat = 2560, k = 1024, SM = prop.multiProcessorCount;
  const tc::GemmPlan p = tc::plan_gemm(n_tok, n_feat, k, false, SM, false);  // (k-split not allowed)
  // the one instantiation that has the withholding compiled in: 16-token epilogue chunks, no k-split, two issuing threads
  if (p.splits != 1 || p.issuers != 2 || ((p.tile_tok & 31) == 0 && p.tile_tok >= 96)) return ADIT_E_UNSUPPORTED;
  auto withhold_kernel = tc::gemm_tc_kernel<false, EPI_STORE_F32, 16, false, 2, true, true>;
  if (cudaFuncSetAttribute(withhold_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BUDGET + 1024) != cudaSuccess) return ADIT_E_CUDA;
  void *a = nullptr, *w = nullptr;
  float* out = nullptr;
  int* status = nullptr;
  const size_t rows_padded = (size_t)p.n_ttiles * p.tile_tok;
  bool ok = cudaMalloc(&a, (size_t)rows_padded * k * 2) == cudaSuccess && cudaMalloc(&w, (size_t)n_feat * k * 2) == cudaSuccess &&
            cudaMalloc((void**)&out, rows_padded * n_feat * 4) == cudaSuccess && cudaMalloc((void**)&status, 4) == cudaSuccess;
  int rc = ADIT_E_CUDA;
  if (ok) {
    cudaMemset(a, 0, rows_padded * k * 2);
    cudaMemset(w, 0, (size_t)n_feat * k * 2);
    cudaMemset(status, 0, 4);
    CUtensorMap mw, ma;
    cudaStream_t st = (cudaStream_t)stream;
    if (tc::make_map_bf16(&mw, w, n_feat, k, tc::TILE_F) && tc::make_map_bf16(&ma, a, rows_padded, k, p.tile_tok)) {
      tc::GemmArgs g{};
      g.n_feat = n_feat; g.n_tok = n_tok; g.epi = EPI_STORE_F32; g.out = out; g.ldo = n_feat; g.status = status;
      g.debug_withhold = 3;
      g.kb_total = p.kb_total; g.tile_tok = p.tile_tok; g.n_ftiles = p.n_ftiles; g.n_ttiles = p.n_ttiles; g.splits = 1;
      g.stages = p.stages; g.tmem_cols = p.tmem_cols; g.ring_bytes = p.ring_bytes; g.acc_bufs = p.acc_bufs; g.issuers = p.issuers;
      withhold_kernel<<<tc::gemm_grid(p, SM), tc::GEMM_THREADS, p.smem_bytes, st>>>(mw, ma, g);
      cudaError_t e = cudaGetLastError();
      if (e == cudaSuccess) e = cudaStreamSynchronize(st);
      int hs = 0;
      if (e == cudaSuccess) e = cudaMemcpy(&hs, status, 4, cudaMemcpyDeviceToHost);
      *first_status = hs;
      if (e == cudaSuccess) {
        cudaMemset(status, 0, 4);
        g.debug_withhold = 0;
        e = tc::launch_gemm(mw, ma, p, false, g, SM, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e == cudaSuccess) e = cudaMemcpy(&hs, status, 4, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess) rc = hs;
      }
      if (e != cudaSuccess) cudaGetLastError();
    }
  }
  if (a) cudaFree(a);
  if (w) cudaFree(w);
  if (out) cudaFree(out);
  if (status) cudaFree(status);
  return rc;
}

// ---------------------------------------------------------------------------------------------
// Streaming-read microbenchmark: what a plain read of global memory reaches from a given number of SMs
// (the HBM denominator for runs on a reduced SM budget).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) stream_read_kernel(const uint4* __restrict__ src, size_t n_vec, unsigned* __restrict__ sink) {
  const size_t per = (n_vec + gridDim.x - 1) / gridDim.x;
  const size_t lo = (size_t)blockIdx.x * per, hi = lo + per < n_vec ? lo + per : n_vec;
  unsigned acc = 0;
  size_t i = lo + threadIdx.x;
  for (; i + 7 * 512 < hi; i += 8 * 512) {
    uint4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v[j].x), "=r"(v[j].y), "=r"(v[j].z), "=r"(v[j].w) : "l"(src + i + (size_t)j * 512));
#pragma unroll
    for (int j = 0; j < 8; ++j) acc ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
  }
  for (; i < hi; i += 512) { const uint4 v = src[i]; acc ^= v.x ^ v.y ^ v.z ^ v.w; }
  if (acc == 0x9e3779b9u) sink[blockIdx.x] = acc;  // (keeps the loads alive; practically never true)
}

extern "C" int adit_debug_stream_read(int device, size_t bytes, int sm_count, int iters, double* gb_per_s) {
  if (!gb_per_s || bytes < (1u << 20) || iters < 1 || sm_count < 1) return ADIT_E_INVALID;
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  void* buf = nullptr; unsigned* sink = nullptr;
  if (cudaMalloc(&buf, bytes) != cudaSuccess) return ADIT_E_CUDA;
  if (cudaMalloc((void**)&sink, 4096 * 4) != cudaSuccess) { cudaFree(buf); return ADIT_E_CUDA; }
  cudaMemset(buf, 1, bytes);
  cudaEvent_t a, b;
  cudaEventCreate(&a); cudaEventCreate(&b);
  const int grid = sm_count > 4096 ? 4096 : sm_count;
  stream_read_kernel<<<grid, 512>>>((const uint4*)buf, bytes / 16, sink);
  cudaEventRecord(a);
  for (int i = 0; i < iters; ++i) stream_read_kernel<<<grid, 512>>>((const uint4*)buf, bytes / 16, sink);
  cudaEventRecord(b);
  cudaError_t e = cudaEventSynchronize(b);
  float ms = 0.f;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
  cudaEventDestroy(a); cudaEventDestroy(b);
  cudaFree(buf); cudaFree(sink);
  if (e != cudaSuccess || ms <= 0.f) return ADIT_E_CUDA;
  *gb_per_s = (double)bytes * iters / (ms * 1e-3) / 1e9;
  return ADIT_OK;
}

// ---------------------------------------------------------------------------------------------
// Background GEMM load (stand-in for the VLM stage on the other stream)
// ---------------------------------------------------------------------------------------------
struct adit_bg_gemm {
  int device, m, n, k, sm_count;
  void *a, *b, *c;
  int* status;
  CUtensorMap map_a, map_b;
  tc::GemmPlan plan;
};

__global__ void bg_fill_kernel(bf16* __restrict__ p, int64_t n, uint32_t seed) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    uint32_t x = (uint32_t)i * 2654435761u + seed;
    x ^= x >> 15; x *= 2246822519u; x ^= x >> 13;
    p[i] = __float2bfloat16_rn(((int)(x & 0xffff) - 32768) * (1.0f / 65536.0f));
  }
}

extern "C" int adit_bg_gemm_create(int device, int m, int n, int k, adit_bg_gemm** out) {
  return adit_bg_gemm_create_kind(device, m, n, k, 0, out);
}

extern "C" int adit_bg_gemm_create_kind(int device, int m, int n, int k, int kind, adit_bg_gemm** out) {
  if (!out || m < 1 || n < 1 || k < 64 || (k % 64) || kind < 0 || kind > 1) return ADIT_E_INVALID;
  if (cudaSetDevice(device) != cudaSuccess) return ADIT_E_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return ADIT_E_CUDA;
  if (prop.major != 10) return ADIT_E_UNSUPPORTED;
  if (tc::ensure_smem_attr() != cudaSuccess) return ADIT_E_CUDA;
  adit_bg_gemm* g = new (std::nothrow) adit_bg_gemm();
  if (!g) return ADIT_E_INVALID;
  g->device = device; g->m = m; g->n = n; g->k = k; g->sm_count = prop.multiProcessorCount;
  g->a = g->b = g->c = nullptr; g->status = nullptr;
  if (kind == 1 && g->sm_count < 2) { delete g; return ADIT_E_UNSUPPORTED; }
  g->plan = kind == 1 ? tc::plan_gemm_pair(m, n, k, false, g->sm_count) : tc::plan_gemm(m, n, k, false, g->sm_count, false);
  const size_t rows_c = (size_t)g->plan.n_ttiles * g->plan.tile_tok;  // whole token tiles are stored
  bool ok = cudaMalloc(&g->a, (size_t)m * k * 2) == cudaSuccess && cudaMalloc(&g->b, (size_t)n * k * 2) == cudaSuccess &&
            cudaMalloc(&g->c, rows_c * n * 2) == cudaSuccess && cudaMalloc((void**)&g->status, 4) == cudaSuccess;
  if (ok) {
    cudaMemset(g->status, 0, 4);
    bg_fill_kernel<<<1024, 256>>>((bf16*)g->a, (int64_t)m * k, 1u);
    bg_fill_kernel<<<1024, 256>>>((bf16*)g->b, (int64_t)n * k, 2u);
    ok = cudaDeviceSynchronize() == cudaSuccess && tc::make_map_bf16(&g->map_a, g->a, m, k, tc::token_box_rows(g->plan)) &&
         tc::make_map_bf16(&g->map_b, g->b, n, k, tc::TILE_F);
  }
  if (!ok) {
    adit_bg_gemm_destroy(g);
    return ADIT_E_CUDA;
  }
  *out = g;
  return ADIT_OK;
}

extern "C" int adit_bg_gemm_launch(adit_bg_gemm* g, int iters, int sm_count, void* stream) {
  if (!g || iters < 0) return ADIT_E_INVALID;
  if (cudaSetDevice(g->device) != cudaSuccess) return ADIT_E_CUDA;
  const int G = (sm_count <= 0 || sm_count >= g->sm_count) ? g->sm_count : sm_count;
  tc::GemmArgs a{};
  a.n_feat = g->n; a.n_tok = g->m; a.epi = EPI_STORE; a.out = g->c; a.ldo = g->n; a.status = g->status;
  for (int i = 0; i < iters; ++i)
    if (tc::launch_gemm(g->map_b, g->map_a, g->plan, false, a, G, (cudaStream_t)stream) != cudaSuccess) return ADIT_E_CUDA;
  return ADIT_OK;
}

extern "C" int adit_bg_gemm_destroy(adit_bg_gemm* g) {
  if (!g) return ADIT_OK;
  cudaSetDevice(g->device);
  cudaDeviceSynchronize();
  if (g->a) cudaFree(g->a);
  if (g->b) cudaFree(g->b);
  if (g->c) cudaFree(g->c);
  if (g->status) cudaFree(g->status);
  delete g;
  return ADIT_OK;
}
