// Shared declarations of the ADiT library: element types, small device helpers, epilogue ids.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace adit {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float silu_f(float y) { return y / (1.0f + __expf(-y)); }
__device__ __forceinline__ float silu_precise(float y) { return y / (1.0f + expf(-y)); }
__device__ __forceinline__ float gelu_tanh_f(float y) {
  const float c = 0.7978845608028654f;  // sqrt(2/pi)
  return 0.5f * y * (1.0f + tanhf(c * (y + 0.044715f * y * y * y)));
}

// Epilogues of the projection kernels (what happens to an accumulator element acc[m][n]).
enum Epilogue : int {
  EPI_STORE = 0,      // out[m][n] = acc * rowscale[m] (if rowscale) + bias[n] (if bias), compute dtype
  EPI_SILU_VEC = 1,   // out[m][n] = silu(acc + vec[n]), compute dtype
  EPI_RESIDUAL = 2,   // outf[m][n] += acc, fp32
  EPI_EMBED_OUT = 3,  // outf[m + m / horizon + 1][n] = acc + bias[n], fp32 (action row -> token row)
  EPI_GEGLU = 4,      // out[m][n] = gelu_tanh(acc_gate * rowscale[m]) * (acc_up * rowscale[m]), compute dtype
  EPI_STORE_F32 = 5   // outf[m][n] = acc + bias[n] (if bias), fp32
};

struct EpiArgs {
  void* out;              // compute dtype or fp32, per epilogue
  int ldo;                // leading dimension of out, in elements
  const float* rowscale;  // [M] or null
  const float* bias;      // [N] or null (EPI_SILU_VEC: the added vector)
  int horizon;            // EPI_EMBED_OUT row mapping
};

// Per-call description of the ragged prefix caches, passed by value as a kernel parameter so that
// the caller's host arrays are consumed at launch.
struct PrefixTable {
  const void* kv[64];
  int32_t len[64];
};

// Per-call tensor maps of the requests' prefix caches for the tensor-core attention kernel: request b's cache seen
// as a 3-D tensor (channel, row, plane = (layer, K|V, kv head)) whose row extent is prefix_len[b], so that rows at or
// beyond it are never read (the copy engine writes zeros for them).  Written to device memory by a small kernel
// from its by-value parameter, like the call descriptor.
struct KvMaps {
  alignas(64) CUtensorMap pk[64];
};

// Everything that changes from one adit_denoise call to the next.  The kernels of the captured launch
// graph read it from device memory; a one-block kernel launched ahead of the graph writes it there
// from its by-value parameter, so the caller's host arrays are consumed at enqueue time.
struct CallDesc {
  PrefixTable pt;
  const float* state;
  const float* noise;
  float* out;
};

}  // namespace adit
