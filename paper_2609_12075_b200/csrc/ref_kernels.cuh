// Plain CUDA kernels (no tensor cores): the fp32 debug path, and small per-call pieces shared by
// both dtypes (prologue, action projection, read-out + Euler update).
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace adit {

// ---------------------------------------------------------------------------------------------
// C[M,N] = epilogue(A[M,K] * W[N,K]^T): 64x64 tile, 16-deep k-slab, 256 threads, 4x4 per thread.
// DUAL: a second weight matrix W2 = W + dual_off rows (gate/up pair) feeds a second accumulator.
// ---------------------------------------------------------------------------------------------
template <typename TA, typename TW, typename TO, int EPI, bool DUAL>
__global__ void __launch_bounds__(256) ref_gemm_kernel(const TA* __restrict__ A, int lda,
                                                       const TW* __restrict__ W, int ldw, int64_t dual_off,
                                                       int gu_block, int M, int N, int K, EpiArgs ea) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  __shared__ float W2s[DUAL ? BK : 1][BN + 4];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tx = tid % 16, ty = tid / 16;
  float acc[4][4] = {}, acc2[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += BK) {
    for (int e = tid; e < BM * BK; e += 256) {
      int r = e / BK, c = e % BK;
      int m = m0 + r, k = k0 + c;
      As[c][r] = (m < M && k < K) ? to_f32(A[(int64_t)m * lda + k]) : 0.f;
      int n = n0 + r;
      float w = 0.f, w2 = 0.f;
      if (n < N && k < K) {
        // gate/up rows are interleaved in blocks of gu_block rows: [gate block | up block] ...
        int64_t row = DUAL ? ((int64_t)(n / gu_block) * 2 * gu_block + n % gu_block) : n;
        w = to_f32(W[row * ldw + k]);
        if (DUAL) w2 = to_f32(W[(row + dual_off) * ldw + k]);
      }
      Ws[c][r] = w;
      if (DUAL) W2s[c][r] = w2;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4], b2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = Ws[kk][tx * 4 + j];
        if (DUAL) b2[j] = W2s[kk][tx * 4 + j];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
          if (DUAL) acc2[i][j] = fmaf(a[i], b2[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    float rs = ea.rowscale ? ea.rowscale[m] : 1.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = acc[i][j];
      if (EPI == EPI_STORE) {
        v = v * rs + (ea.bias ? ea.bias[n] : 0.f);
        ((TO*)ea.out)[(int64_t)m * ea.ldo + n] = from_f32<TO>(v);
      } else if (EPI == EPI_SILU_VEC) {
        ((TO*)ea.out)[(int64_t)m * ea.ldo + n] = from_f32<TO>(silu_precise(v + ea.bias[n]));
      } else if (EPI == EPI_RESIDUAL) {
        ((float*)ea.out)[(int64_t)m * ea.ldo + n] += v;
      } else if (EPI == EPI_EMBED_OUT) {
        int row = m + m / ea.horizon + 1;
        ((float*)ea.out)[(int64_t)row * ea.ldo + n] = v + ea.bias[n];
      } else if (EPI == EPI_GEGLU) {
        ((TO*)ea.out)[(int64_t)m * ea.ldo + n] = from_f32<TO>(gelu_tanh_f(v * rs) * (acc2[i][j] * rs));
      } else if (EPI == EPI_STORE_F32) {
        ((float*)ea.out)[(int64_t)m * ea.ldo + n] = v + (ea.bias ? ea.bias[n] : 0.f);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Row statistics of the residual stream: rstd[m] = 1/sqrt(mean(h[m]^2) + eps), hb[m] = T(h[m]).
// (The norm gain is folded into the rows of the following weight matrix, so the projection of
// the normalised row is  rstd[m] * (h[m] . (g * W)).)
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) rowstats_kernel(const float* __restrict__ h, T* __restrict__ hb,
                                                       float* __restrict__ rstd, int D, float eps) {
  const int m = blockIdx.x;
  const float* row = h + (int64_t)m * D;
  float ss = 0.f;
  for (int d = threadIdx.x; d < D; d += blockDim.x) {
    float v = row[d];
    ss = fmaf(v, v, ss);
    hb[(int64_t)m * D + d] = from_f32<T>(v);
  }
  __shared__ float red[8];
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    rstd[m] = 1.0f / sqrtf(t / (float)D + eps);
  }
}

// ---------------------------------------------------------------------------------------------
// Ragged-prefix attention, one block per (suffix token, query head, request); 4 warps stride over
// the keys [prefix 0..P_b) ++ [suffix 0..N) with an online softmax, then merge.
// Rows at or beyond prefix_len are never addressed.
// ---------------------------------------------------------------------------------------------
template <typename T, int DH>
__global__ void __launch_bounds__(128) ref_attention_kernel(const T* __restrict__ qkv, int ldqkv, T* __restrict__ att,
                                                            int ldatt, PrefixTable pt, int layer, int n_tokens,
                                                            int n_q_heads, int n_kv_heads, int p_cap, float scale,
                                                            int state_mask) {
  constexpr int E = DH / 32;
  const int tok = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
  const int kvh = hq / (n_q_heads / n_kv_heads);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int plen = pt.len[b];
  const int total = plen + n_tokens;
  const int64_t row0 = (int64_t)b * n_tokens;
  const T* qrow = qkv + (row0 + tok) * ldqkv + hq * DH;
  const int k_off = n_q_heads * DH + kvh * DH;
  const int v_off = k_off + n_kv_heads * DH;
  const T* pk = (const T*)pt.kv[b] + ((int64_t)(layer * 2 + 0) * n_kv_heads + kvh) * p_cap * DH;
  const T* pv = (const T*)pt.kv[b] + ((int64_t)(layer * 2 + 1) * n_kv_heads + kvh) * p_cap * DH;
  float q[E], acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    q[e] = to_f32(qrow[lane + 32 * e]);
    acc[e] = 0.f;
  }
  float mx = -INFINITY, l = 0.f;
  for (int key = warp; key < total; key += 4) {
    if (state_mask && tok == 0 && key > plen) break;  // the state token sees the prefix and itself only
    const T *kr, *vr;
    if (key < plen) {
      kr = pk + (int64_t)key * DH;
      vr = pv + (int64_t)key * DH;
    } else {
      const T* r = qkv + (row0 + (key - plen)) * ldqkv;
      kr = r + k_off;
      vr = r + v_off;
    }
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) s = fmaf(q[e], to_f32(kr[lane + 32 * e]), s);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    s *= scale;
    float mn = fmaxf(mx, s);
    float corr = expf(mx - mn), p = expf(s - mn);
    l = l * corr + p;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = fmaf(p, to_f32(vr[lane + 32 * e]), acc[e] * corr);
    mx = mn;
  }
  __shared__ float s_m[4], s_l[4], s_acc[4][DH];
  if (lane == 0) { s_m[warp] = mx; s_l[warp] = l; }
#pragma unroll
  for (int e = 0; e < E; ++e) s_acc[warp][lane + 32 * e] = acc[e];
  __syncthreads();
  float M = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
  float wgt[4], L = 0.f;
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    wgt[w] = (s_m[w] == -INFINITY) ? 0.f : expf(s_m[w] - M);
    L += s_l[w] * wgt[w];
  }
  for (int d = threadIdx.x; d < DH; d += 128) {
    float o = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) o += s_acc[w][d] * wgt[w];
    att[(row0 + tok) * ldatt + hq * DH + d] = from_f32<T>(o / L);
  }
}

// ---------------------------------------------------------------------------------------------
// Prologue pieces (once per call).
// ---------------------------------------------------------------------------------------------
// tau[k][j]: sinusoidal embedding of t_k = k/K, computed in fp64 and stored fp32.
__global__ void time_table_kernel(float* __restrict__ tau, int n_steps, int dim, double pmin, double pmax) {
  const int half = dim / 2;
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_steps * half) return;
  int k = idx / half, j = idx % half;
  double t = (double)k / (double)n_steps;
  double period = pmin * pow(pmax / pmin, (double)j / (double)(half - 1));
  double ang = 2.0 * 3.14159265358979323846 * t / period;
  tau[(int64_t)k * dim + j] = (float)sin(ang);
  tau[(int64_t)k * dim + half + j] = (float)cos(ang);
}

// x <- noise;  hs[b][n] = state[b] . Ws[n][:] + bs[n]
// (desc, when given, supplies the call's noise and state pointers.)
__global__ void prologue_kernel(const CallDesc* __restrict__ desc, const float* __restrict__ noise,
                                float* __restrict__ x, int n_x, const float* __restrict__ state,
                                const float* __restrict__ Ws, const float* __restrict__ bs, float* __restrict__ hs,
                                int B, int S, int D) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();
  if (desc) { noise = desc->noise; state = desc->state; }
  const int n_max = n_x > B * D ? n_x : B * D;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < n_max; idx += gridDim.x * blockDim.x) {
    if (idx < n_x) x[idx] = noise[idx];
    if (idx < B * D) {
      int b = idx / D, n = idx % D;
      float a = bs[n];
      for (int j = 0; j < S; ++j) a = fmaf(state[b * S + j], Ws[(int64_t)n * S + j], a);
      hs[idx] = a;
    }
  }
}

// Per step: ea[m][n] = T(x[m] . Wa[n][:] + ba[n]) for the action rows; state rows of h <- hs.
template <typename T>
__global__ void embed_in_kernel(const float* __restrict__ x, const float* __restrict__ Wa, const float* __restrict__ ba,
                                T* __restrict__ ea, const float* __restrict__ hs, float* __restrict__ h, int B,
                                int horizon, int A, int D) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();
  const int64_t n_act = (int64_t)B * horizon * D;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n_act;
       idx += (int64_t)gridDim.x * blockDim.x) {
    int m = (int)(idx / D), n = (int)(idx % D);
    float a = ba[n];
    for (int j = 0; j < A; ++j) a = fmaf(x[(int64_t)m * A + j], Wa[(int64_t)n * A + j], a);
    ea[idx] = from_f32<T>(a);
    if (idx < (int64_t)B * D) {
      int b = (int)(idx / D);
      h[((int64_t)b * (horizon + 1)) * D + n] = hs[idx];
    }
  }
}

// Read-out and Euler update, one block (256 threads) per action row (or per row and part of the outputs when
// `parts` > 1: small batches get more blocks that way; every part recomputes the row's 1/rms):
//   v = (h_row * rstd) . Wout'[j][:] + bout[j]   (final-norm gain folded into Wout'),  x += dt * v.
// The row is staged in shared memory; each warp takes outputs j = warp, warp + 8, ... and reads the
// weight row with 128-bit loads.  D must be a multiple of 4.
__global__ void __launch_bounds__(256) final_kernel(const float* __restrict__ h, const float* __restrict__ Wout,
                                                    const float* __restrict__ bout, float* __restrict__ x,
                                                    float* __restrict__ out, int horizon, int A, int D, float eps,
                                                    float dt, int n_rows, int parts,
                                                    const CallDesc* __restrict__ desc) {
  extern __shared__ float4 srow[];  // D / 4
  __shared__ float red[8];
  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();
  if (desc) out = desc->out;  // last step of a call whose output pointer lives in the call descriptor
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int per_part = (A + parts - 1) / parts;
  for (int item = blockIdx.x; item < n_rows * parts; item += gridDim.x) {
    const int m = item / parts, part = item - m * parts;  // action row b*horizon + i, and which outputs
    const int j_end = min(A, (part + 1) * per_part);
    const float4* row = reinterpret_cast<const float4*>(h + ((int64_t)m + m / horizon + 1) * D);
    float ss = 0.f;
    __syncthreads();
    for (int d = threadIdx.x; d < D / 4; d += 256) {
      float4 v = row[d];
      srow[d] = v;
      ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) red[warp] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float rstd = 1.0f / sqrtf(tot / (float)D + eps);
    for (int j = part * per_part + warp; j < j_end; j += 8) {
      const float4* wr = reinterpret_cast<const float4*>(Wout + (int64_t)j * D);
      float a = 0.f;
      for (int d = lane; d < D / 4; d += 32) {
        const float4 w4 = __ldg(wr + d), v = srow[d];
        a = fmaf(v.x, w4.x, a); a = fmaf(v.y, w4.y, a); a = fmaf(v.z, w4.z, a); a = fmaf(v.w, w4.w, a);
      }
      for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      if (lane == 0) {
        float xn = x[(int64_t)m * A + j] + dt * (a * rstd + bout[j]);
        x[(int64_t)m * A + j] = xn;
        if (out) out[(int64_t)m * A + j] = xn;
      }
    }
  }
}


// ---------------------------------------------------------------------------------------------
// Rotary embedding on the suffix queries and keys (variant ADIT_FLAG_SUFFIX_ROPE).
// Once per call: cos/sin of pos * 10000^(-2j/dh) for every suffix token row, pos = prefix_len[b] + index in the
// suffix, computed in fp64 and kept as fp32 pairs [row][dh/2].  After every Q/K/V projection: channel pairs
// (j, j + dh/2) of every query head and key head of the row are rotated in place.
// ---------------------------------------------------------------------------------------------
__global__ void rope_table_kernel(float2* __restrict__ tab, PrefixTable pt, const PrefixTable* __restrict__ ptp, int n_rows,
                                  int n_tokens, int dh) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();
  const int half = dh / 2;
  const PrefixTable& t = ptp ? *ptp : pt;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < (int64_t)n_rows * half; i += (int64_t)gridDim.x * blockDim.x) {
    const int row = (int)(i / half), j = (int)(i % half);
    const int b = row / n_tokens;
    const double pos = (double)(t.len[b] + (row - b * n_tokens));
    const double ang = pos * pow(10000.0, -(double)j / (double)half);
    tab[i] = make_float2((float)cos(ang), (float)sin(ang));
  }
}

template <typename T>
__global__ void __launch_bounds__(128) rope_apply_kernel(T* __restrict__ qkv, int ldqkv, const float2* __restrict__ tab, int n_rows,
                                                         int n_rot_heads, int dh) {
  ptx::pdl_launch_dependents();
  ptx::pdl_wait_prior_grids();
  const int half = dh / 2;
  const int64_t n = (int64_t)n_rows * n_rot_heads * half;   // query heads then key heads are contiguous in a row
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int j = (int)(i % half);
    const int hd = (int)((i / half) % n_rot_heads);
    const int row = (int)(i / ((int64_t)half * n_rot_heads));
    T* p = qkv + (int64_t)row * ldqkv + hd * dh;
    const float2 cs = tab[(int64_t)row * half + j];
    const float x1 = to_f32(p[j]), x2 = to_f32(p[j + half]);
    p[j] = from_f32<T>(x1 * cs.x - x2 * cs.y);
    p[j + half] = from_f32<T>(x2 * cs.x + x1 * cs.y);
  }
}

// ---------------------------------------------------------------------------------------------
// Weight packing (load time): dst[(row_off + map(o))][i] = T(src[i][o] * gain[i]) from a row-major
// [n_in, n_out] fp32 source; map interleaves gate/up rows in blocks when gu_block > 0.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void pack_rows_kernel(const float* __restrict__ src, int n_in, int n_out, const float* __restrict__ gain,
                                 T* __restrict__ dst, int64_t row_off, int ld, int gu_block, int gu_second) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n_in * n_out) return;
  int o = (int)(idx / n_in), i = (int)(idx % n_in);
  float v = src[(int64_t)i * n_out + o];
  if (gain) v *= gain[i];
  int64_t r = o;
  if (gu_block > 0) r = (int64_t)(o / gu_block) * 2 * gu_block + o % gu_block + (gu_second ? gu_block : 0);
  dst[(row_off + r) * ld + i] = from_f32<T>(v);
}

__global__ void set_desc_kernel(CallDesc d, CallDesc* __restrict__ dst) {
  if (threadIdx.x == 0) *dst = d;
}

__global__ void bf16_bits_to_f32_kernel(const uint16_t* __restrict__ src, float* __restrict__ dst, int64_t n) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < n) dst[idx] = __uint_as_float(((uint32_t)src[idx]) << 16);
}

}  // namespace adit
