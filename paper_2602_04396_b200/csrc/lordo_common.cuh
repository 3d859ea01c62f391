// Shared device-side definitions of the LoRDO hot path (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lordo.h"

namespace lordo {

// ---------------------------------------------------------------------------------------------
// Per-matrix device record, built once by lordo_init and kept in the workspace.
// ---------------------------------------------------------------------------------------------
struct MatDev {
  long long m, n;     // storage shape of W, G, E, X0, B, Delta
  int r;
  int side;           // 1: projected from the right, handled as the left-side problem on the transpose
  long long pm, ln;   // rows of P and columns of the low-rank arrays: (m, n), or (n, m) for side 1
  void* W;            // [K][m][n] w_dtype
  void* E;            // [K][m][n] e_dtype
  float* P;           // [pm][r] or [K][pm][r]
  float* u;           // [K][r][ln]
  float* v;           // [K][r][ln]
  float* X0;          // [m][n]
  float* B;           // [m][n]
  float* Delta;       // [m][n]
  float* ghat;        // [K][r][ln] low-rank gradient (workspace)
  float* util;        // [K][r][ln] normalised low-rank update U~ (workspace)
  float* dcol;        // [K][ln]   column scale of the full-rank QHM term (workspace)
  long long p_stride; // elements between the P of consecutive replicas (0 for Global)
  __nv_bfloat16* Delta16;  // [m][n] bf16 copy of Delta, made at the start of a Global refresh for the tensor-core sketch (workspace; may be null)
  float* T;           // [K][r][ln] up-link time buffer: sum over the round of lr * U~ (workspace; null unless enabled)
};

// Scalars of one inner step (Algorithm 1, per-step lines).
struct StepScalars {
  float lr, beta1, beta2, omega, eps;
  float inv_bc1, inv_bc2;  // 1/(1-beta1^s), 1/(1-beta2^s)
  int form;                // lordo_qhm
  int ef;                  // error feedback on
  int K;
};

// ---------------------------------------------------------------------------------------------
// Element access: fp32 or bf16 storage, fp32 arithmetic.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_bits_to_float(unsigned short b) { return __uint_as_float(((unsigned)b) << 16); }

__device__ __forceinline__ float4 load4(const void* base, int dt, long long idx) {
  if (dt == LORDO_F32) {
    return *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + idx);
  }
  uint2 raw = *reinterpret_cast<const uint2*>(reinterpret_cast<const unsigned short*>(base) + idx);
  float4 o;
  o.x = __uint_as_float(raw.x << 16);
  o.y = __uint_as_float(raw.x & 0xFFFF0000u);
  o.z = __uint_as_float(raw.y << 16);
  o.w = __uint_as_float(raw.y & 0xFFFF0000u);
  return o;
}

__device__ __forceinline__ float load1(const void* base, int dt, long long idx) {
  if (dt == LORDO_F32) return reinterpret_cast<const float*>(base)[idx];
  return bf16_bits_to_float(reinterpret_cast<const unsigned short*>(base)[idx]);
}

__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);  // round to nearest even
  return *reinterpret_cast<unsigned*>(&h);
}

__device__ __forceinline__ void store4(void* base, int dt, long long idx, float4 v) {
  if (dt == LORDO_F32) {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(base) + idx) = v;
  } else {
    uint2 raw;
    raw.x = pack_bf16x2(v.x, v.y);
    raw.y = pack_bf16x2(v.z, v.w);
    *reinterpret_cast<uint2*>(reinterpret_cast<unsigned short*>(base) + idx) = raw;
  }
}

__device__ __forceinline__ void store1(void* base, int dt, long long idx, float v) {
  if (dt == LORDO_F32) {
    reinterpret_cast<float*>(base)[idx] = v;
  } else {
    __nv_bfloat16 h = __float2bfloat16_rn(v);
    reinterpret_cast<__nv_bfloat16*>(base)[idx] = h;
  }
}

// Largest index i in [0, count) with start[i] <= x (start is ascending, start[0] == 0).
__device__ __forceinline__ int find_segment(const long long* __restrict__ start, int count, long long x) {
  int lo = 0, hi = count - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (start[mid] <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// ---------------------------------------------------------------------------------------------
// Counter-based generator for P_0 and the sketches (integers only).
// ---------------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ unsigned long long mix64(unsigned long long x) {
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
constexpr unsigned long long kGolden = 0x9E3779B97F4A7C15ull;

__host__ __device__ inline unsigned long long stream_key(unsigned long long seed, int purpose, int mat, long long index, int replica) {
  unsigned long long k = mix64(seed + kGolden);
  const unsigned long long f[4] = {(unsigned long long)purpose, (unsigned long long)mat, (unsigned long long)index,
                                   (unsigned long long)replica};
  for (int i = 0; i < 4; ++i) k = mix64(k + kGolden * (f[i] + 1ull));
  return k;
}

}  // namespace lordo
