// Ragged-prefix attention on tensor cores (bf16 in, fp32 accumulate).
//
// For request b and kv head kvh, the G = n_q_heads / n_kv_heads query heads that share the kv head
// and the N suffix tokens form one dense block of R = N * G query rows (row r -> token r / G, head
// kvh * G + r % G) against the key list [prefix 0..P_b) ++ [suffix 0..N).  A work item is
// (request, kv head, tile of 16 * NW query rows, key split); it streams 64-key blocks of K and V
// through shared memory (cp.async, rows outside the valid key list are written as zeros and masked
// to -inf, so padding rows of the caller's cache are never read), computes S = Q K^T and O += P V
// with mma.sync m16n8k16 and keeps the softmax online in registers (row max / row sum reduced across
// the four lanes of a quad with shuffles; exp2 with log2(e)/sqrt(dh) folded into the scale).
// With more than one key split the unnormalised partial (O, m, l) goes to a workspace and a merge
// kernel combines the splits in fixed order.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace adit {
namespace attn {

constexpr int KEY_BLOCK = 64;

struct AttnArgs {
  const bf16* qkv;  // [M, ldqkv]: Q heads, then K heads, then V heads
  int ldqkv;
  bf16* att;        // [M, ldatt]
  int ldatt;
  int layer, n_tokens, n_q_heads, n_kv_heads, p_cap, batch;
  int n_row_tiles;  // ceil(N * G / (16 * NW))
  int splits;
  float scale_log2; // log2(e) / sqrt(dh)
  void* part_o;     // [splits][M * n_q_heads][DH] (splits > 1): fp32 from the mma.sync kernel, bf16 from the tcgen05 kernel
  float* part_ml;   // [splits][M * n_q_heads][2]
  unsigned long long* trace;  // optional [grid][4]: block start, predecessor-wait released, end (%globaltimer ns)
  int q_tma;        // tcgen05 kernel: the query tile comes in by TMA (group size divides 128)
  unsigned long long* dbg;  // optional [grid][16] phase stamps of the tcgen05 kernel (test aid)
  int* status;      // device-visible status word (ADIT_E_TIMEOUT = -6 on an expired wait); may be null
  const CUtensorMap* kv_maps;  // tcgen05 kernel: per-request tensor maps of the prefix caches (device memory, see KvMaps)
  int state_mask;   // variant: the first suffix token of a request attends to the prefix and itself only
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                                  const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void mma_bf16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int DH, int NW>
__global__ void __launch_bounds__(32 * NW) attn_mma_kernel(AttnArgs a, const PrefixTable* __restrict__ ptp) {
  ptx::pdl_launch_dependents();
  if (a.trace && threadIdx.x == 0) a.trace[blockIdx.x * 4] = ptx::globaltimer_ns();
  ptx::pdl_wait_prior_grids();
  const PrefixTable& pt = *ptp;
  constexpr int ROWS = 16 * NW;
  constexpr int LDS = DH + 8;          // padded row (elements): 16 extra bytes keep ldmatrix conflict-free
  constexpr int CHUNKS = DH / 8;       // 16-byte chunks per row
  extern __shared__ __align__(16) uint8_t smem[];
  bf16* sQ = reinterpret_cast<bf16*>(smem);
  bf16* sK = sQ + ROWS * LDS;
  bf16* sV = sK + KEY_BLOCK * LDS;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = a.n_q_heads / a.n_kv_heads;
  const int R = a.n_tokens * G;
  const int k_off = a.n_q_heads * DH, v_off = k_off + a.n_kv_heads * DH;
  const int n_items = a.batch * a.n_kv_heads * a.n_row_tiles * a.splits;

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    int t = item;
    const int split = t % a.splits; t /= a.splits;
    const int rt = t % a.n_row_tiles; t /= a.n_row_tiles;
    const int kvh = t % a.n_kv_heads;
    const int b = t / a.n_kv_heads;
    const int plen = pt.len[b];
    const int total = plen + a.n_tokens;
    const int nkb = (total + KEY_BLOCK - 1) / KEY_BLOCK;
    const int kb0 = (int)((int64_t)split * nkb / a.splits), kb1 = (int)((int64_t)(split + 1) * nkb / a.splits);
    const int64_t tok0 = (int64_t)b * a.n_tokens;
    const bf16* pk = (const bf16*)pt.kv[b] + ((int64_t)(a.layer * 2 + 0) * a.n_kv_heads + kvh) * a.p_cap * DH;
    const bf16* pv = (const bf16*)pt.kv[b] + ((int64_t)(a.layer * 2 + 1) * a.n_kv_heads + kvh) * a.p_cap * DH;

    __syncthreads();  // the previous item's readers of sQ/sK/sV are done
    // ---- Q tile ----
    for (int e = tid; e < ROWS * CHUNKS; e += 32 * NW) {
      const int r = e / CHUNKS, c = e % CHUNKS;
      const int gr = rt * ROWS + r;
      bf16* dst = sQ + r * LDS + c * 8;
      if (gr < R) {
        const int tok = gr / G, hq = kvh * G + gr % G;
        cp_async16(dst, a.qkv + (tok0 + tok) * a.ldqkv + hq * DH + c * 8);
      } else {
        *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
      }
    }
    cp_async_commit();

    float o[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // rows lane/4 and lane/4 + 8 of this warp

    for (int kb = kb0; kb < kb1; ++kb) {
      __syncthreads();  // everyone finished reading the previous K/V block
      for (int e = tid; e < KEY_BLOCK * CHUNKS; e += 32 * NW) {
        const int r = e / CHUNKS, c = e % CHUNKS;
        const int key = kb * KEY_BLOCK + r;
        bf16* dk = sK + r * LDS + c * 8;
        bf16* dv = sV + r * LDS + c * 8;
        if (key < plen) {
          cp_async16(dk, pk + (int64_t)key * DH + c * 8);
          cp_async16(dv, pv + (int64_t)key * DH + c * 8);
        } else if (key < total) {
          const bf16* row = a.qkv + (tok0 + (key - plen)) * a.ldqkv;
          cp_async16(dk, row + k_off + kvh * DH + c * 8);
          cp_async16(dv, row + v_off + kvh * DH + c * 8);
        } else {
          *reinterpret_cast<uint4*>(dk) = make_uint4(0, 0, 0, 0);
          *reinterpret_cast<uint4*>(dv) = make_uint4(0, 0, 0, 0);
        }
      }
      cp_async_commit();
      cp_async_wait_all();
      __syncthreads();

      // ---- S = Q K^T for this warp's 16 rows x 64 keys ----
      float s[8][4];
#pragma unroll
      for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks) {
        uint32_t a0, a1, a2, a3;
        ldmatrix_x4(a0, a1, a2, a3, sQ + (warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDS + ks * 16 + (lane >> 4) * 8);
#pragma unroll
        for (int np = 0; np < 4; ++np) {  // pairs of 8-key tiles
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(b0, b1, b2, b3, sK + (np * 16 + (lane & 7) + (lane >> 4) * 8) * LDS + ks * 16 + ((lane >> 3) & 1) * 8);
          mma_bf16(s[2 * np], a0, a1, a2, a3, b0, b1);
          mma_bf16(s[2 * np + 1], a0, a1, a2, a3, b2, b3);
        }
      }
      // ---- scale, mask, online softmax ----
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int key = kb * KEY_BLOCK + nt * 8 + (lane & 3) * 2;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool valid = (key + (e & 1)) < total;
          s[nt][e] = valid ? s[nt][e] * a.scale_log2 : -INFINITY;
        }
        mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
        mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);  // finite: every block holds a valid key
      const float c0 = exp2f(m0 - mn0), c1 = exp2f(m1 - mn1);
      m0 = mn0; m1 = mn1;
      float rs0 = 0.f, rs1 = 0.f;
      uint32_t pa[4][4];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const float p0 = exp2f(s[nt][0] - mn0), p1 = exp2f(s[nt][1] - mn0);
        const float p2 = exp2f(s[nt][2] - mn1), p3 = exp2f(s[nt][3] - mn1);
        rs0 += p0 + p1;
        rs1 += p2 + p3;
        pa[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
        pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      l0 = l0 * c0 + rs0;  // per-lane partial row sums; reduced across the quad at the end
      l1 = l1 * c1 + rs1;
#pragma unroll
      for (int i = 0; i < DH / 8; ++i) {
        o[i][0] *= c0; o[i][1] *= c0; o[i][2] *= c1; o[i][3] *= c1;
      }
      // ---- O += P V ----
#pragma unroll
      for (int j = 0; j < 4; ++j) {  // 16 keys per k-step
#pragma unroll
        for (int dp = 0; dp < DH / 16; ++dp) {  // pairs of 8-wide d tiles
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(b0, b1, b2, b3, sV + (j * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDS + dp * 16 + (lane >> 4) * 8);
          mma_bf16(o[2 * dp], pa[j][0], pa[j][1], pa[j][2], pa[j][3], b0, b1);
          mma_bf16(o[2 * dp + 1], pa[j][0], pa[j][1], pa[j][2], pa[j][3], b2, b3);
        }
      }
    }
    if (kb0 >= kb1) {
      cp_async_wait_all();
    }
    // ---- finish: row sums across the quad, then store ----
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int gr = rt * ROWS + warp * 16 + (lane >> 2) + half * 8;
      if (gr >= R) continue;
      const int tok = gr / G, hq = kvh * G + gr % G;
      const float l = half ? l1 : l0, m = half ? m1 : m0;
      if (a.splits == 1) {
        const float inv = 1.0f / l;
        bf16* dst = a.att + (tok0 + tok) * a.ldatt + hq * DH + (lane & 3) * 2;
#pragma unroll
        for (int i = 0; i < DH / 8; ++i)
          *reinterpret_cast<uint32_t*>(dst + i * 8) = pack_bf16(o[i][half * 2] * inv, o[i][half * 2 + 1] * inv);
      } else {
        const int64_t qrow = (tok0 + tok) * a.n_q_heads + hq;
        const int64_t n_qrows = (int64_t)a.batch * a.n_tokens * a.n_q_heads;
        float* dst = (float*)a.part_o + ((int64_t)split * n_qrows + qrow) * DH + (lane & 3) * 2;
#pragma unroll
        for (int i = 0; i < DH / 8; ++i)
          *reinterpret_cast<float2*>(dst + i * 8) = make_float2(o[i][half * 2], o[i][half * 2 + 1]);
        if ((lane & 3) == 0) {
          float* ml = a.part_ml + ((int64_t)split * n_qrows + qrow) * 2;
          ml[0] = m;
          ml[1] = l;
        }
      }
    }
  }
  if (a.trace && threadIdx.x == 0) a.trace[blockIdx.x * 4 + 2] = ptx::globaltimer_ns();
}

// Merge of key splits, fixed order: one warp per query row; each lane owns DH / 32 contiguous
// channels.  Loads of up to four splits are in flight at a time; the additions stay in split order.
// TP is the element type of the partial outputs: float (mma.sync kernel) or bf16 (tcgen05 kernel).
// HV = 2 (bf16 partials, DH >= 128): a warp takes half of a row's channels, which halves the chain of dependent
// instructions per warp; the (m, l) work is repeated by both halves.
template <int DH, typename TP, int NB = 4, int HV = 1>
__global__ void __launch_bounds__(128) attn_merge_kernel(const TP* __restrict__ part_o,
                                                         const float* __restrict__ part_ml, int splits,
                                                         int64_t n_qrows, int n_q_heads, bf16* __restrict__ att,
                                                         int ldatt, unsigned long long* trace) {
  ptx::pdl_launch_dependents();
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4] = ptx::globaltimer_ns();
  ptx::pdl_wait_prior_grids();
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4 + 1] = ptx::globaltimer_ns();
  constexpr int E = DH / 32;  // 2, 4 or 8 contiguous floats per lane
  const int lane = threadIdx.x & 31;
  static_assert(HV == 1 || (sizeof(TP) == 2 && DH >= 128), "half rows: bf16 partials of at least 128 channels");
  for (int64_t u = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5); u < n_qrows * HV; u += (int64_t)gridDim.x * 4) {
    const int64_t q = u / HV;
    const int ch0 = (int)(u % HV) * (DH / HV) + lane * (E / HV);  // this lane's first channel
    // lane s keeps (m, l) of split s (splits <= 32 by construction)
    float my_m = -INFINITY, my_l = 0.f;
    if (lane < splits) {
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml + (lane * n_qrows + q) * 2));
      my_m = ml.x; my_l = ml.y;
    }
    if constexpr (sizeof(TP) == 2) {
      // bf16 partials: the loads of up to NB splits are issued before anything depends on the (m, l) pairs, so
      // a row with few splits costs about one round trip to L2 (NB = 16 is used for more than 4 splits)
      constexpr int W = E / HV / 2;  // 32-bit words per lane and split
      float accb[2 * W];
#pragma unroll
      for (int e = 0; e < 2 * W; ++e) accb[e] = 0.f;
      float Mb = my_m;
      float Lb = 0.f, wb = 0.f;
      for (int s0 = 0; s0 < splits; s0 += NB) {
        uint32_t raw[NB][W];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
          if (s0 + i < splits) {
            const TP* po = part_o + ((s0 + i) * n_qrows + q) * DH + ch0;
            if constexpr (W == 1) {
              raw[i][0] = __ldcg(reinterpret_cast<const uint32_t*>(po));
            } else if constexpr (W == 2) {
              const uint2 t = __ldcg(reinterpret_cast<const uint2*>(po));
              raw[i][0] = t.x; raw[i][1] = t.y;
            } else {
              const uint4 t = __ldcg(reinterpret_cast<const uint4*>(po));
              raw[i][0] = t.x; raw[i][1] = t.y; raw[i][2] = t.z; raw[i][3] = t.w;
            }
          }
        }
        if (s0 == 0) {
          for (int o = 16; o; o >>= 1) Mb = fmaxf(Mb, __shfl_xor_sync(0xffffffffu, Mb, o));
          wb = (my_m == -INFINITY) ? 0.f : exp2f(my_m - Mb);
          // (lanes without a split hold l = 0: a butterfly over all lanes, the same total in every lane)
          Lb = my_l * wb;
          for (int o = 16; o; o >>= 1) Lb += __shfl_xor_sync(0xffffffffu, Lb, o);
        }
#pragma unroll
        for (int i = 0; i < NB; ++i) {
          if (s0 + i < splits) {
            const float w = __shfl_sync(0xffffffffu, wb, s0 + i);
#pragma unroll
            for (int k = 0; k < W; ++k) {
              accb[2 * k] = fmaf(__uint_as_float(raw[i][k] << 16), w, accb[2 * k]);
              accb[2 * k + 1] = fmaf(__uint_as_float(raw[i][k] & 0xffff0000u), w, accb[2 * k + 1]);
            }
          }
        }
      }
      const float invb = 1.0f / Lb;
      const int64_t tokb = q / n_q_heads;
      const int hqb = (int)(q % n_q_heads);
      bf16* dstb = att + tokb * ldatt + hqb * DH + ch0;
#pragma unroll
      for (int e = 0; e < 2 * W; e += 2)
        *reinterpret_cast<uint32_t*>(dstb + e) = pack_bf16(accb[e] * invb, accb[e + 1] * invb);
      continue;
    }
    float M = my_m;
    for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    const float my_w = (my_m == -INFINITY) ? 0.f : exp2f(my_m - M);
    float L = 0.f;
    for (int s = 0; s < splits; ++s) L += __shfl_sync(0xffffffffu, my_l * my_w, s);
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (int s0 = 0; s0 < splits; s0 += 4) {
      float v[4][E];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (s0 + i < splits) {
          const TP* po = part_o + ((s0 + i) * n_qrows + q) * DH + lane * E;
          if constexpr (sizeof(TP) == 2) {  // bf16: E * 2 bytes per lane
            if constexpr (E == 2) {
              const uint32_t t = __ldcg(reinterpret_cast<const uint32_t*>(po));
              v[i][0] = __uint_as_float(t << 16); v[i][1] = __uint_as_float(t & 0xffff0000u);
            } else if constexpr (E == 4) {
              const uint2 t = __ldcg(reinterpret_cast<const uint2*>(po));
              v[i][0] = __uint_as_float(t.x << 16); v[i][1] = __uint_as_float(t.x & 0xffff0000u);
              v[i][2] = __uint_as_float(t.y << 16); v[i][3] = __uint_as_float(t.y & 0xffff0000u);
            } else {
              const uint4 t = __ldcg(reinterpret_cast<const uint4*>(po));
              v[i][0] = __uint_as_float(t.x << 16); v[i][1] = __uint_as_float(t.x & 0xffff0000u);
              v[i][2] = __uint_as_float(t.y << 16); v[i][3] = __uint_as_float(t.y & 0xffff0000u);
              v[i][4] = __uint_as_float(t.z << 16); v[i][5] = __uint_as_float(t.z & 0xffff0000u);
              v[i][6] = __uint_as_float(t.w << 16); v[i][7] = __uint_as_float(t.w & 0xffff0000u);
            }
          } else if constexpr (E == 2) {
            float2 t = __ldcg(reinterpret_cast<const float2*>(po));
            v[i][0] = t.x; v[i][1] = t.y;
          } else {
#pragma unroll
            for (int e = 0; e < E; e += 4) {
              float4 t = __ldcg(reinterpret_cast<const float4*>(po + e));
              v[i][e] = t.x; v[i][e + 1] = t.y; v[i][e + 2] = t.z; v[i][e + 3] = t.w;
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (s0 + i < splits) {
          const float w = __shfl_sync(0xffffffffu, my_w, s0 + i);
#pragma unroll
          for (int e = 0; e < E; ++e) acc[e] = fmaf(v[i][e], w, acc[e]);
        }
      }
    }
    const float inv = 1.0f / L;
    const int64_t tok = q / n_q_heads;
    const int hq = (int)(q % n_q_heads);
    bf16* dst = att + tok * ldatt + hq * DH + lane * E;
#pragma unroll
    for (int e = 0; e < E; e += 2)
      *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16(acc[e] * inv, acc[e + 1] * inv);
  }
  if (trace && threadIdx.x == 0) trace[blockIdx.x * 4 + 2] = ptx::globaltimer_ns();
}

template <int DH, int NW>
constexpr size_t attn_smem_bytes() {
  return (size_t)(16 * NW + 2 * KEY_BLOCK) * (DH + 8) * 2;
}

}  // namespace attn
}  // namespace adit
